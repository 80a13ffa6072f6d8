"""Plain fp64 CPU oracle of the action-conditioned batched decode step.

TEST INFRASTRUCTURE.  This file defines what the CUDA library must compute.
It is deliberately slow and literal: NumPy in float64, one sequence / one
head at a time, library calls (matmul, lexsort, exp) as single steps, no
blocking, fusion or reordering.  It shares no code with the CUDA path and
must never be imported by the product package.

Every sequence i of the batch carries its own efficiency action, the paper's
tuple (kappa, rho, q) ("Actions and controlled compute", Method section),
renamed here as in the benchmark spec:

    r = kappa   attention keep-rate,   passed as r_permille in [0, 1000]
    p = 1-rho   MLP prune rate,        passed as p_permille in [0, 1000]
    b = q       activation bit-width,  2..8 or 16

Rates are per-mille integers so that every count is an exact integer formula.

Readings taken where the paper is silent or the benchmark spec overrides it:

  * quantizer rounding is round-to-nearest-even; an all-zero row gives
    scale 0 and codes 0; the arithmetic that decides a code is IEEE fp32
    (scale = a / q_max, then x / scale), so codes can be bit-exact;
  * b = 16 is bf16 passthrough (the paper: "q >= 16 returns the input
    unchanged");
  * the quantizer is applied to the inputs of the QKV and gate/up
    projections (the task's default placement); the paper's own placement,
    the MLP output before the residual add, is PLACE_MLP_OUTPUT, and widths
    of 9..15 bits (int16 codes) are supported in both;
  * token selection is exact top-k per (sequence, kv-head) on the q.k score
    summed over the query group (the paper uses Quest page bounds per head);
    forced-keep tokens (sinks, recent window; default: only the newest
    token) count toward the budget; softmax runs over the kept set only;
  * MLP pruning drops the p fraction of *intermediate* channels with the
    smallest |silu(g)*u| per token (the task's default); the paper's own
    form, gating the MLP block's input channels by |x|, is PRUNE_MLP_INPUT;
    the kept count mirrors the paper's ceil form in both;
  * the paper's own selection, SELECT_QUEST_PAGES (quest_decode_attn): pages
    of S contiguous tokens from token 0, extrema of a partial last page over
    the keys that exist, top ceil(b_t / S) pages per QUERY head, the page of
    the newest token always among them, every key of a kept page attended;
  * ties are broken toward the lower index;
  * T (seq_lens) counts the newest token, whose k/v the layer appends
    before attention reads the cache.

Parity status: every function below is pinned by tests that do not go
through this file's own arithmetic (dense library references, brute force
over subsets, closed forms, hand-computed fixtures).  The paper prints no
worked numeric example, so no fixture carries paper-printed values.

bf16 tensors are numpy uint16 arrays holding the bit patterns.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

# ----------------------------------------------------------------------------
# bf16 <-> float64 (storage format only; no method arithmetic here)
# ----------------------------------------------------------------------------


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float64, exactly."""
    u = np.asarray(u16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bf16 (ties to even), in ONE rounding.

    Works on the float64 bit pattern: bf16 keeps 7 of the 52 fraction bits.
    Valid for zeros and for magnitudes inside bf16's normal range, which is
    all this oracle produces; anything else raises.
    """
    x = np.ascontiguousarray(x, dtype=np.float64)
    ax = np.abs(x)
    ok = (ax == 0) | ((ax >= 2.0 ** -126) & (ax < 2.0 ** 127))
    if not np.all(ok):
        raise ValueError("value outside the bf16 normal range")
    bits = x.view(np.uint64)
    drop = np.uint64(45)
    lsb = (bits >> drop) & np.uint64(1)
    rounded = bits + (np.uint64((1 << 44) - 1) + lsb)
    rounded = (rounded >> drop) << drop
    as_f32 = rounded.view(np.float64).astype(np.float32)  # exact: 8 significant bits
    return (as_f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def f32_to_bf16_rne(x32: np.ndarray) -> np.ndarray:
    """Round float32 to bf16, ties to even (exact widening, then one rounding)."""
    return f64_to_bf16_rne(np.asarray(x32, dtype=np.float32).astype(np.float64))


# ----------------------------------------------------------------------------
# Shapes and containers
# ----------------------------------------------------------------------------


@dataclass
class Shape:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    page_size: int = 64
    rms_eps: float = 1e-5
    rope_theta: float = 0.0  # 0 = no rotary embedding
    n_sink: int = 0
    n_window: int = 1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass
class LayerWeights:
    """bf16 bit patterns.  w_qkv rows: all q heads, then k heads, then v heads."""

    w_qkv: np.ndarray  # [(Hq+2Hkv)*hd][d]
    w_o: np.ndarray  # [d][Hq*hd]
    w_gate: np.ndarray  # [ff][d]
    w_up: np.ndarray  # [ff][d]
    w_down_t: np.ndarray  # [ff][d]   row j = intermediate channel j
    gamma1: np.ndarray  # [d]
    gamma2: np.ndarray  # [d]


@dataclass
class PagedKV:
    k_pool: np.ndarray  # uint16 [num_pages][Hkv][page][hd]
    v_pool: np.ndarray
    page_table: np.ndarray  # int32 [B][max_pages_per_seq]
    seq_lens: np.ndarray  # int32 [B], valid tokens INCLUDING the newest


# ----------------------------------------------------------------------------
# Counts
# ----------------------------------------------------------------------------


def forced_keep_set(T: int, n_sink: int, n_window: int) -> np.ndarray:
    """Indices that are always attended: the first n_sink and the last n_window
    tokens (the paper's always-dense sink / window tokens, Method section,
    "Policy inputs and architecture").  The task's default is n_sink = 0,
    n_window = 1: only the newest token."""
    f = set(range(min(max(n_sink, 0), T))) | set(range(max(T - max(n_window, 0), 0), T))
    return np.array(sorted(f), dtype=np.int64)


def kept_token_count(r_permille: int, T: int, n_forced: int) -> int:
    """Token budget b_t = ceil(kappa_t * K_t), clamped to [0, K_t] (appendix on
    efficiency actions, "Budgeted token selection"), then raised to the number
    of forced tokens so the newest token is always kept."""
    if not 0 <= r_permille <= 1000:
        raise ValueError("r_permille out of range")
    b = (int(r_permille) * int(T) + 999) // 1000
    b = min(max(b, 0), T)
    return min(T, max(b, n_forced))


def kept_channel_count(p_permille: int, ff: int) -> int:
    """Kept intermediate channels m = ceil((1 - p) * ff); mirrors the paper's
    m_t = ceil(rho_t * d) ("Per-token channel selection") with rho = 1 - p."""
    if not 0 <= p_permille <= 1000:
        raise ValueError("p_permille out of range")
    return ((1000 - int(p_permille)) * int(ff) + 999) // 1000


# ----------------------------------------------------------------------------
# Activation quantization
# ----------------------------------------------------------------------------


def quantize_per_token(x32: np.ndarray, bits: int):
    """Per-token symmetric quantizer (appendix "Activation quantization",
    "Quantizer"): q_max = 2^(b-1) - 1, a = max_j |x_j|, s = a / q_max,
    code_j = clip(round(x_j / s), -q_max, q_max), x_hat_j = code_j * s.

    x32 is one token's float32 vector.  Both divisions are IEEE float32 and
    the rounding is to nearest-even.  Returns (codes, scale float32, x_hat
    float64); codes are int8 up to 8 bits and int16 from 9 to 15 bits (the
    paper's action tables use widths up to 15).  bits == 16: passthrough to
    bf16; codes are all zero and scale is 1.
    """
    x32 = np.asarray(x32, dtype=np.float32)
    if bits == 16:
        xh = bf16_to_f64(f32_to_bf16_rne(x32))
        return np.zeros(x32.shape, np.int8), np.float32(1.0), xh
    if not 2 <= bits <= 15:
        raise ValueError("unsupported bit-width")
    ctype = np.int8 if bits <= 8 else np.int16
    q_max = (1 << (bits - 1)) - 1
    a = np.float32(np.max(np.abs(x32))) if x32.size else np.float32(0)
    if a == 0:
        return np.zeros(x32.shape, ctype), np.float32(0.0), np.zeros(x32.shape, np.float64)
    s = np.float32(a) / np.float32(q_max)  # IEEE fp32 division
    ratio = (x32 / s).astype(np.float32)  # IEEE fp32 division, element-wise
    c = np.clip(np.rint(ratio), -q_max, q_max)
    codes = c.astype(ctype)
    x_hat = codes.astype(np.float64) * np.float64(s)
    return codes, np.float32(s), x_hat


def fake_quant_mlp_output(z: np.ndarray, bits: int):
    """The paper's own placement of the quantizer (appendix "Activation
    quantization", "What is quantized"): the MLP block's output z, the update
    of the residual stream, is quantized and dequantized per token before it is
    added back; the matmuls themselves run at full precision.  Same operator as
    quantize_per_token on fl32(z); from 16 bits on z is returned unchanged
    ("For q >= 16 we return z unchanged": no rounding at all in this placement).
    Returns (codes, scale float32, z_hat float64)."""
    z = np.asarray(z, np.float64)
    if bits >= 16:
        return np.zeros(z.shape, np.int16), np.float32(1.0), z.copy()
    return quantize_per_token(z.astype(np.float32), bits)


def quant_act(x_bf16: np.ndarray, bits: Sequence[int]):
    """Batched form over bf16 rows: what the stand-alone quantize call returns."""
    x_bf16 = np.asarray(x_bf16, dtype=np.uint16)
    B, d = x_bf16.shape
    codes = np.zeros((B, d), np.int16 if any(8 < int(b) < 16 for b in bits) else np.int8)
    scales = np.zeros(B, np.float32)
    x_hat = np.zeros((B, d), np.float64)
    for i in range(B):
        x32 = bf16_to_f64(x_bf16[i]).astype(np.float32)
        codes[i], scales[i], x_hat[i] = quantize_per_token(x32, int(bits[i]))
    return codes, scales, x_hat


# ----------------------------------------------------------------------------
# RMSNorm and rotary embedding (the frozen LLaMA layer around the actions)
# ----------------------------------------------------------------------------


def rmsnorm(h: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """x_j = h_j * gamma_j / sqrt(mean_j h_j^2 + eps), float64."""
    h = np.asarray(h, np.float64)
    return h * np.asarray(gamma, np.float64) / math.sqrt(float(np.mean(h * h)) + eps)


def rope_rotate(vec: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary embedding in the rotate-half convention: element i pairs with
    element i + hd/2, angle pos * theta^(-2i/hd).  theta == 0 disables it."""
    v = np.asarray(vec, np.float64)
    if theta == 0:
        return v.copy()
    hd = v.shape[-1]
    half = hd // 2
    i = np.arange(half, dtype=np.float64)
    ang = float(pos) * np.power(float(theta), -2.0 * i / hd)
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = v[..., :half], v[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


# ----------------------------------------------------------------------------
# Selection
# ----------------------------------------------------------------------------


def select_top(score: np.ndarray, k: int, forced: np.ndarray) -> np.ndarray:
    """The forced indices plus the k - |forced| non-forced indices with the
    largest score; order of preference (score descending, index ascending).
    Returns the kept indices in ascending order."""
    score = np.asarray(score, np.float64)
    n = score.shape[0]
    forced = np.asarray(forced, np.int64)
    assert len(forced) <= k <= n
    free = np.ones(n, bool)
    free[forced] = False
    cand = np.nonzero(free)[0]
    order = np.lexsort((cand, -score[cand]))  # primary: score desc; secondary: index asc
    chosen = cand[order[: k - len(forced)]]
    return np.sort(np.concatenate([forced, chosen])).astype(np.int64)


# ----------------------------------------------------------------------------
# Attention with a per-sequence keep-rate
# ----------------------------------------------------------------------------


def cache_rows(pool: np.ndarray, page_table_row: np.ndarray, T: int, kvh: int) -> np.ndarray:
    """Tokens 0..T-1 of one kv-head of one sequence, as float64 [T][hd]."""
    P = pool.shape[2]
    n_pages = (T + P - 1) // P
    rows = np.concatenate([pool[int(page_table_row[pg]), kvh] for pg in range(n_pages)], axis=0)[:T]
    return bf16_to_f64(rows)


def sparse_attention_one_group(q_group: np.ndarray, K: np.ndarray, V: np.ndarray, k_keep: int,
                               forced: np.ndarray):
    """One (sequence, kv-head): q_group [G][hd], K and V [T][hd], all float64.

    Selection score sigma_j = sum_h q_h . k_j (unscaled); kept set by
    select_top; then, per query head, softmax over the kept logits
    q_h . k_j / sqrt(hd) only (the paper's additive -inf mask on dropped
    keys, "Quest masking in LLaMA attention") and the weighted sum of the
    kept v rows."""
    G, hd = q_group.shape
    dots = K @ q_group.T  # [T][G]
    sigma = dots.sum(axis=1)
    kept = select_top(sigma, k_keep, forced)
    logits = dots[kept] / math.sqrt(hd)  # [k][G]
    out = np.zeros((G, hd))
    for h in range(G):
        z = logits[:, h] - logits[:, h].max()
        w = np.exp(z)
        w /= w.sum()
        out[h] = w @ V[kept]
    return out, kept, sigma


def sparse_decode_attn(shape: Shape, q: np.ndarray, kv: PagedKV, r_permille: Sequence[int]):
    """q float64 [B][Hq][hd] (already rotated).  Returns out float64
    [B][Hq][hd], kept[i][kvh] index arrays and sigma[i][kvh] score arrays."""
    B = q.shape[0]
    G = shape.group
    out = np.zeros((B, shape.n_q_heads, shape.head_dim))
    kept_all: List[List[np.ndarray]] = []
    sigma_all: List[List[np.ndarray]] = []
    for i in range(B):
        T = int(kv.seq_lens[i])
        forced = forced_keep_set(T, shape.n_sink, shape.n_window)
        k_keep = kept_token_count(int(r_permille[i]), T, len(forced))
        kept_i, sigma_i = [], []
        for kvh in range(shape.n_kv_heads):
            K = cache_rows(kv.k_pool, kv.page_table[i], T, kvh)
            V = cache_rows(kv.v_pool, kv.page_table[i], T, kvh)
            o, kept, sigma = sparse_attention_one_group(q[i, kvh * G:(kvh + 1) * G], K, V, k_keep, forced)
            out[i, kvh * G:(kvh + 1) * G] = o
            kept_i.append(kept)
            sigma_i.append(sigma)
        kept_all.append(kept_i)
        sigma_all.append(sigma_i)
    return out, kept_all, sigma_all


# ----------------------------------------------------------------------------
# The paper's own token sparsity: Quest page selection per query head
# (appendix on efficiency actions, "Token sparsity via Quest": "Budgeted token
# selection", "Quest masking in LLaMA attention", "Granularity")
# ----------------------------------------------------------------------------
SELECT_TOKENS = 0       # the task's default: exact top-k tokens per (sequence, kv-head) (sparse_decode_attn)
SELECT_QUEST_PAGES = 1  # the paper's: top pages per query head by the Quest bound (quest_decode_attn)


def quest_page_extrema(K: np.ndarray, S: int):
    """K float64 [T][hd] -> (m_plus, m_minus), each [ceil(T/S)][hd]: per-dimension
    m+ = max_j k_j and m- = -min_j k_j over the keys of each page of S contiguous
    tokens.  The last page may hold fewer than S keys; the padding the paper adds
    is masked there, so here the extrema run over the keys that exist."""
    T = K.shape[0]
    P = (T + S - 1) // S
    m_plus = np.stack([K[pg * S:min((pg + 1) * S, T)].max(axis=0) for pg in range(P)])
    m_minus = np.stack([-K[pg * S:min((pg + 1) * S, T)].min(axis=0) for pg in range(P)])
    return m_plus, m_minus


def quest_page_scores(q: np.ndarray, m_plus: np.ndarray, m_minus: np.ndarray) -> np.ndarray:
    """score(page) = q_pos . m+ + q_neg . m-, with q_pos = |q| * [q >= 0] and
    q_neg = |q| - q_pos (one query head, q float64 [hd])."""
    a = np.abs(q)
    q_pos = a * (q >= 0)
    q_neg = a - q_pos
    return m_plus @ q_pos + m_minus @ q_neg


def quest_kept_page_count(r_permille: int, T: int, S: int, n_forced_pages: int) -> int:
    """ceil(b_t / S) pages with b_t = ceil(kappa_t K_t) clamped to [0, K_t], never
    more than there are pages, never fewer than the forced ones (the page of the
    newest token, so that the step always attends to it)."""
    if not 0 <= r_permille <= 1000:
        raise ValueError("r_permille out of range")
    b = min(max((int(r_permille) * int(T) + 999) // 1000, 0), T)
    P = (T + S - 1) // S
    return min(P, max((b + S - 1) // S, n_forced_pages))


def quest_attention_one_group(q_group: np.ndarray, K: np.ndarray, V: np.ndarray, S: int, n_keep: int,
                              forced_pages: np.ndarray):
    """One (sequence, kv-head): every query head of the group picks its own
    n_keep pages (forced ones first, then by score descending, page index
    ascending), attends to all keys of its pages and to nothing else (additive
    -inf on the others) with logits q . k / sqrt(hd).  Returns out [G][hd], the
    kept page indices per head (ascending) and the scores [G][pages]."""
    G, hd = q_group.shape
    T = K.shape[0]
    m_plus, m_minus = quest_page_extrema(K, S)
    out = np.zeros((G, hd))
    kept_pages, scores = [], []
    for h in range(G):
        sc = quest_page_scores(q_group[h], m_plus, m_minus)
        pages = select_top(sc, n_keep, forced_pages)
        tok = np.concatenate([np.arange(pg * S, min((pg + 1) * S, T)) for pg in pages])
        logit = K[tok] @ q_group[h] / math.sqrt(hd)
        w = np.exp(logit - logit.max())
        w /= w.sum()
        out[h] = w @ V[tok]
        kept_pages.append(pages)
        scores.append(sc)
    return out, kept_pages, np.stack(scores)


def quest_decode_attn(shape: Shape, q: np.ndarray, kv: PagedKV, r_permille: Sequence[int], S: int):
    """q float64 [B][Hq][hd] (already rotated).  Returns out float64 [B][Hq][hd],
    kept_pages[i][query head] and scores[i][query head] (per-page bounds)."""
    B = q.shape[0]
    G = shape.group
    out = np.zeros((B, shape.n_q_heads, shape.head_dim))
    kept_all, score_all = [], []
    for i in range(B):
        T = int(kv.seq_lens[i])
        forced_tok = forced_keep_set(T, shape.n_sink, shape.n_window)
        forced_pages = np.unique(forced_tok // S)
        n_keep = quest_kept_page_count(int(r_permille[i]), T, S, len(forced_pages))
        kept_i, score_i = [], []
        for kvh in range(shape.n_kv_heads):
            K = cache_rows(kv.k_pool, kv.page_table[i], T, kvh)
            V = cache_rows(kv.v_pool, kv.page_table[i], T, kvh)
            o, pages, sc = quest_attention_one_group(q[i, kvh * G:(kvh + 1) * G], K, V, S, n_keep, forced_pages)
            out[i, kvh * G:(kvh + 1) * G] = o
            kept_i.extend(pages)
            score_i.extend(list(sc))
        kept_all.append(kept_i)
        score_all.append(score_i)
    return out, kept_all, score_all


# ----------------------------------------------------------------------------
# SwiGLU MLP with a per-token prune rate
# ----------------------------------------------------------------------------


def silu(g: np.ndarray) -> np.ndarray:
    return g / (1.0 + np.exp(-g))


def pruned_swiglu_mlp(x_hat: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down_t: np.ndarray,
                      p_permille: Sequence[int]):
    """x_hat float64 [B][d]; weights bf16 bit patterns.  Per token:
    g = W_g x, u = W_u x, t_j = silu(g_j) u_j, keep the m = ceil((1-p) ff)
    channels with the largest |t_j|, out = sum over kept j of t_j W_down[j, :].
    Returns out float64 [B][d], kept channel arrays, t float64 [B][ff]."""
    Wg, Wu, Wd = bf16_to_f64(w_gate), bf16_to_f64(w_up), bf16_to_f64(w_down_t)
    ff = Wg.shape[0]
    B = x_hat.shape[0]
    out = np.zeros((B, Wd.shape[1]))
    t_all = np.zeros((B, ff))
    kept_all = []
    none = np.zeros(0, np.int64)
    for i in range(B):
        g = Wg @ x_hat[i]
        u = Wu @ x_hat[i]
        t = silu(g) * u
        m = kept_channel_count(int(p_permille[i]), ff)
        kept = select_top(np.abs(t), m, none)
        out[i] = t[kept] @ Wd[kept]
        t_all[i] = t
        kept_all.append(kept)
    return out, kept_all, t_all


# ----------------------------------------------------------------------------
# One decoder layer, and a stack of them
# ----------------------------------------------------------------------------


@dataclass
class LayerTrace:
    xn1: Optional[np.ndarray] = None  # float32 [B][d] normalised attention input
    codes1: Optional[np.ndarray] = None
    scales1: Optional[np.ndarray] = None
    q_rot: Optional[np.ndarray] = None  # float64 [B][Hq][hd]
    k_new: Optional[np.ndarray] = None  # uint16 [B][Hkv][hd] as appended
    v_new: Optional[np.ndarray] = None
    kept_tokens: Optional[list] = None
    attn_out: Optional[np.ndarray] = None
    h_mid: Optional[np.ndarray] = None  # float64 [B][d]
    xn2: Optional[np.ndarray] = None
    codes2: Optional[np.ndarray] = None
    scales2: Optional[np.ndarray] = None
    t: Optional[np.ndarray] = None
    kept_channels: Optional[list] = None
    extra: Dict[str, np.ndarray] = field(default_factory=dict)


def norm_and_quantize(h: np.ndarray, gamma_bf16: np.ndarray, eps: float, bits: Sequence[int]):
    """RMSNorm in float64, cast to float32, then the per-token quantizer."""
    B, d = h.shape
    gamma = bf16_to_f64(gamma_bf16)
    xn = np.zeros((B, d), np.float32)
    codes = np.zeros((B, d), np.int16 if any(8 < int(b) < 16 for b in bits) else np.int8)
    scales = np.zeros(B, np.float32)
    x_hat = np.zeros((B, d))
    for i in range(B):
        xn[i] = rmsnorm(h[i], gamma, eps).astype(np.float32)
        codes[i], scales[i], x_hat[i] = quantize_per_token(xn[i], int(bits[i]))
    return xn, codes, scales, x_hat


def append_kv(shape: Shape, kv: PagedKV, i: int, k_bf16: np.ndarray, v_bf16: np.ndarray) -> None:
    """Write the newest token's k, v ([Hkv][hd] bf16) at position T_i - 1."""
    pos = int(kv.seq_lens[i]) - 1
    page = int(kv.page_table[i, pos // shape.page_size])
    slot = pos % shape.page_size
    kv.k_pool[page, :, slot, :] = k_bf16
    kv.v_pool[page, :, slot, :] = v_bf16


PRUNE_INTERMEDIATE = 0  # the task's default: intermediate channels by |silu(g) u| (pruned_swiglu_mlp)
PRUNE_MLP_INPUT = 1     # the paper's: input channels of the MLP block by |x| (gate_input_channels)


def gate_input_channels(x32: np.ndarray, p_permille: int):
    """The paper's structured MLP pruning (appendix "Structured MLP activation pruning", "Per-token channel
    selection"): of the MLP block's input x (one token, d_model channels) keep the m = ceil(rho * d_model)
    channels of largest magnitude |x(j)|, rho = 1 - p, and zero the rest (a multiplicative 0/1 mask).
    Ties go to the lower index.  The magnitudes are compared as the float32 numbers the quantizer also sees.
    Returns (kept indices ascending, masked x float32)."""
    x32 = np.asarray(x32, np.float32)
    m = kept_channel_count(int(p_permille), x32.shape[0])
    kept = select_top(np.abs(x32).astype(np.float64), m, np.zeros(0, np.int64))
    out = np.zeros_like(x32)
    out[kept] = x32[kept]
    return kept, out


PLACE_PROJ_INPUTS = 0  # the task's default: the inputs of the QKV and gate/up projections are quantized
PLACE_MLP_OUTPUT = 1   # the paper's: the MLP output is fake-quantized before the residual add


def decode_layer(shape: Shape, w: LayerWeights, kv: PagedKV, h_in: np.ndarray,
                 r_permille: Sequence[int], p_permille: Sequence[int], bits: Sequence[int],
                 placement: int = PLACE_PROJ_INPUTS, mlp_prune: int = PRUNE_INTERMEDIATE,
                 token_select: int = SELECT_TOKENS, quest_page_size: int = 16):
    """One decoder layer for one new token per sequence.

    mlp_prune == PRUNE_MLP_INPUT: p_permille[i] gates the input channels of the
    MLP block (gate_input_channels on the normalised row, before the quantizer;
    the attention input of the layer is not pruned) and every intermediate
    channel is kept.

    placement == PLACE_MLP_OUTPUT: the projections read the normalised rows
    through the 16-bit passthrough (bf16, the operand type of the matmuls) and
    bits[i] acts on the MLP output instead (fake_quant_mlp_output).

    h_in float64 [B][d].  kv is modified in place (the newest token's k and v,
    rounded to bf16, are written before attention reads the cache).  No other
    rounding happens between the steps.  Returns (h_out float64 [B][d], trace).
    """
    B, d = h_in.shape
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    tr = LayerTrace()

    in_bits = bits if placement == PLACE_PROJ_INPUTS else [16] * B
    # attention input: RMSNorm, quantize, QKV projection
    tr.xn1, tr.codes1, tr.scales1, x_hat = norm_and_quantize(h_in, w.gamma1, shape.rms_eps, in_bits)
    qkv = x_hat @ bf16_to_f64(w.w_qkv).T  # [B][(Hq+2Hkv)*hd]
    q = qkv[:, : Hq * hd].reshape(B, Hq, hd)
    k = qkv[:, Hq * hd:(Hq + Hkv) * hd].reshape(B, Hkv, hd)
    v = qkv[:, (Hq + Hkv) * hd:].reshape(B, Hkv, hd)

    # rotary embedding at the newest position, then commit k, v to the cache
    q_rot = np.zeros_like(q)
    tr.k_new = np.zeros((B, Hkv, hd), np.uint16)
    tr.v_new = np.zeros((B, Hkv, hd), np.uint16)
    for i in range(B):
        pos = int(kv.seq_lens[i]) - 1
        q_rot[i] = rope_rotate(q[i], pos, shape.rope_theta)
        tr.k_new[i] = f64_to_bf16_rne(rope_rotate(k[i], pos, shape.rope_theta))
        tr.v_new[i] = f64_to_bf16_rne(v[i])
        append_kv(shape, kv, i, tr.k_new[i], tr.v_new[i])
    tr.q_rot = q_rot

    # attention over the kept tokens, output projection, residual
    if token_select == SELECT_QUEST_PAGES:  # the paper's page selection per query head; kept_tokens then holds pages
        attn, tr.kept_tokens, sig = quest_decode_attn(shape, q_rot, kv, r_permille, quest_page_size)
    else:
        attn, tr.kept_tokens, sig = sparse_decode_attn(shape, q_rot, kv, r_permille)
    tr.attn_out = attn
    tr.extra["sigma"] = sig
    h_mid = h_in + attn.reshape(B, Hq * hd) @ bf16_to_f64(w.w_o).T
    tr.h_mid = h_mid

    # MLP input: RMSNorm, quantize; pruned SwiGLU; residual
    if mlp_prune == PRUNE_MLP_INPUT:
        gamma2 = bf16_to_f64(w.gamma2)
        tr.xn2 = np.zeros((B, d), np.float32)
        tr.codes2 = np.zeros((B, d), np.int16 if any(8 < int(b) < 16 for b in in_bits) else np.int8)
        tr.scales2 = np.zeros(B, np.float32)
        x_hat2 = np.zeros((B, d))
        kept_in = []
        for i in range(B):
            tr.xn2[i] = rmsnorm(h_mid[i], gamma2, shape.rms_eps).astype(np.float32)
            kept_i, masked = gate_input_channels(tr.xn2[i], int(p_permille[i]))
            kept_in.append(kept_i)
            tr.codes2[i], tr.scales2[i], x_hat2[i] = quantize_per_token(masked, int(in_bits[i]))
        tr.extra["kept_inputs"] = kept_in
        mlp, tr.kept_channels, tr.t = pruned_swiglu_mlp(x_hat2, w.w_gate, w.w_up, w.w_down_t, [0] * B)
    else:
        tr.xn2, tr.codes2, tr.scales2, x_hat2 = norm_and_quantize(h_mid, w.gamma2, shape.rms_eps, in_bits)
        mlp, tr.kept_channels, tr.t = pruned_swiglu_mlp(x_hat2, w.w_gate, w.w_up, w.w_down_t, p_permille)
    if placement == PLACE_MLP_OUTPUT:
        tr.extra["z"] = mlp.copy()
        z_codes, z_scales = [], np.zeros(B, np.float32)
        for i in range(B):
            c, z_scales[i], mlp[i] = fake_quant_mlp_output(mlp[i], int(bits[i]))
            z_codes.append(c)
        tr.extra["z_codes"], tr.extra["z_scales"] = z_codes, z_scales
    return h_mid + mlp, tr


def decode_step(shape: Shape, layers: Sequence[LayerWeights], kvs: Sequence[PagedKV], h_in_bf16: np.ndarray,
                r_permille, p_permille, bits, placement: int = PLACE_PROJ_INPUTS, mlp_prune: int = PRUNE_INTERMEDIATE):
    """L layers with the same action tuple in every layer (the paper broadcasts
    one action across all layers at a decode step).  The residual stream is
    not rounded between layers.  Returns (h_out float64, [trace per layer])."""
    h = bf16_to_f64(h_in_bf16)
    traces = []
    for w, kv in zip(layers, kvs):
        h, tr = decode_layer(shape, w, kv, h, r_permille, p_permille, bits, placement, mlp_prune)
        traces.append(tr)
    return h, traces


# ----------------------------------------------------------------------------
# Periodic KV-cache refresh (Background, paragraph "Episodes and control
# horizon"): after a horizon of decode steps a fully dense pass over the last
# n_tokens already-known tokens rebuilds their cache entries; no token is
# sampled.
# ----------------------------------------------------------------------------


def kv_refresh(shape: Shape, layers: Sequence[LayerWeights], kvs: Sequence[PagedKV], h_in_bf16: np.ndarray):
    """Dense causal pass over the last n tokens of every sequence, layer by layer.

    h_in_bf16 uint16 [B][n][d]: the layer-0 inputs of the span, oldest first.
    kvs[l].seq_lens counts the span.  In layer l, span token i (position
    T - n + i) is one dense decode_layer row whose context ends at its own
    position: it appends its k, v there and attends to everything before, the
    span tokens j < i of this layer included (they were rewritten just before),
    so the stale entries of tokens j > i are never read.  Dense means keep-rate
    1, prune rate 0, 16 bits.  kvs are modified in place; returns the last
    layer's outputs, float64 [B][n][d]."""
    B, n, d = h_in_bf16.shape
    h = bf16_to_f64(h_in_bf16)
    r, p, b = [1000] * B, [0] * B, [16] * B
    for w, kv in zip(layers, kvs):
        full = np.asarray(kv.seq_lens).copy()
        assert np.all(full >= n), "a sequence is shorter than the refreshed span"
        out = np.zeros_like(h)
        for i in range(n):
            kv.seq_lens = (full - n + 1 + i).astype(np.int32)
            out[:, i], _ = decode_layer(shape, w, kv, h[:, i], r, p, b)
        kv.seq_lens = full
        h = out
    return h
