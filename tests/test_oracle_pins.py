"""Pins for the CPU oracle: each test checks oracle/sol_oracle.py against
something that does not go through its own arithmetic: hand-worked fixtures,
closed forms, brute force over subsets, torch library routines in float64,
and invariants of the definitions.  CPU only."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import sol_oracle as O
from paper_2605_10875_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split(";")]


def t64(u16):
    return torch.from_numpy(O.bf16_to_f64(u16))


# ---------------------------------------------------------------- bf16 ------


def test_bf16_roundtrip_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10 ** rng.uniform(-6, 6, 20000),
                        [0.0, 1.0, -1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e-5, 65504.0]])
    got = O.f64_to_bf16_rne(x)
    # torch rounds float32 -> bf16 to nearest-even; feed it values exactly representable in float32
    x32 = x.astype(np.float32)
    got32 = O.f32_to_bf16_rne(x32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got32, ref)
    # widening is exact and inverts rounding
    assert np.array_equal(O.f64_to_bf16_rne(O.bf16_to_f64(ref)), ref)
    # direct float64 rounding is the NEAREST bf16: no bf16 neighbour is closer
    nz = x != 0  # (the bit pattern below zero's is a NaN)
    x, got = x[nz], got[nz]
    back = O.bf16_to_f64(got)
    up = O.bf16_to_f64((got + 1).astype(np.uint16))
    dn = O.bf16_to_f64((got - 1).astype(np.uint16))
    assert np.all(np.abs(back - x) <= np.abs(up - x))
    assert np.all(np.abs(back - x) <= np.abs(dn - x))


def test_bf16_ties_to_even():
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: goes to the even mantissa (1.0)
    assert O.bf16_to_f64(O.f64_to_bf16_rne(np.array([1.0 + 2.0 ** -8])))[0] == 1.0
    # 1 + 3*2^-8 is halfway between 1+2^-7 (odd) and 1+2^-6 (even)
    assert O.bf16_to_f64(O.f64_to_bf16_rne(np.array([1.0 + 3 * 2.0 ** -8])))[0] == 1.0 + 2.0 ** -6
    # a float64 just above the tie must round up even though float32 would first land on the tie
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert O.bf16_to_f64(O.f64_to_bf16_rne(np.array([x])))[0] == 1.0 + 2.0 ** -7


# --------------------------------------------------------------- counts -----


def test_kept_counts_golden():
    n = 0
    for kind, rate, size, forced, want in _rows("kept_counts.txt"):
        if kind == "token":
            assert O.kept_token_count(int(rate), int(size), int(forced)) == int(want)
        else:
            assert O.kept_channel_count(int(rate), int(size)) == int(want)
        n += 1
    assert n >= 20


def test_kept_counts_closed_form():
    for T in [1, 2, 63, 64, 65, 511, 512, 4096, 8192, 16384, 32768]:
        for r in list(range(0, 1001, 25)) + [1, 125, 999]:
            want = min(T, max(1, math.ceil(Fraction(r, 1000) * T)))
            assert O.kept_token_count(r, T, 1) == want
    for ff in [11, 1024, 8192, 14336]:
        for p in list(range(0, 1001, 50)) + [125, 999]:
            assert O.kept_channel_count(p, ff) == math.ceil(Fraction(1000 - p, 1000) * ff)


def test_forced_set():
    assert list(O.forced_keep_set(10, 0, 1)) == [9]
    assert list(O.forced_keep_set(10, 4, 2)) == [0, 1, 2, 3, 8, 9]
    assert list(O.forced_keep_set(3, 4, 2)) == [0, 1, 2]
    assert list(O.forced_keep_set(5, 0, 0)) == []


# ------------------------------------------------------------ quantizer -----


def test_quantizer_golden():
    n = 0
    for bits, xs, scale, codes in _rows("quantizer_cases.txt"):
        x = np.array([float(v) for v in xs.split()], np.float32)
        c, s, xh = O.quantize_per_token(x, int(bits))
        assert list(c) == [int(v) for v in codes.split()], (bits, xs)
        assert float(s) == float(scale)
        assert np.array_equal(xh, c.astype(np.float64) * float(scale))
        n += 1
    assert n >= 9


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8, 9, 11, 12, 15])
def test_quantizer_properties(bits):
    rng = np.random.default_rng(bits)
    q_max = 2 ** (bits - 1) - 1
    for trial in range(20):
        x = (rng.standard_normal(257) * 10 ** rng.uniform(-3, 3)).astype(np.float32)
        c, s, xh = O.quantize_per_token(x, bits)
        assert c.dtype == (np.int8 if bits <= 8 else np.int16) and np.abs(c.astype(np.int64)).max() <= q_max
        # the scale is the correctly rounded quotient a / q_max
        a = float(np.abs(x).max())
        assert abs(float(s) - a / q_max) <= 2.0 ** -24 * a / q_max
        # reconstruction error at most half a step (plus float32 rounding of x/s: up to q_max * 2^-24 of a step)
        assert np.all(np.abs(x.astype(np.float64) - xh) <= 0.5 * float(s) * (1 + 2e-5) + float(s) * q_max * 2.0 ** -23)
        # the largest-magnitude element maps to +-q_max
        j = int(np.argmax(np.abs(x)))
        assert abs(int(c[j])) == q_max and np.sign(c[j]) == np.sign(x[j])
        # power-of-two rescaling leaves the codes unchanged and scales s
        c2, s2, _ = O.quantize_per_token(x * np.float32(8.0), bits)
        assert np.array_equal(c, c2) and float(s2) == 8.0 * float(s)
        # sign symmetry
        c3, s3, _ = O.quantize_per_token(-x, bits)
        assert np.array_equal(c3, -c) and s3 == s


def test_quantizer_rounds_half_to_even_not_away():
    # q_max = 7, a = 7 -> s = 1: codes are rint(x)
    x = np.array([7, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 6.5], np.float32)
    c, s, _ = O.quantize_per_token(x, 4)
    assert list(c) == [7, 0, 2, 2, 0, -2, -2, 6]


def test_quantizer_passthrough_16_bits():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(1000).astype(np.float32)
    c, s, xh = O.quantize_per_token(x, 16)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(xh, ref) and float(s) == 1.0 and not c.any()
    # a bf16 input is returned unchanged ("q >= 16 returns the input unchanged")
    xb = synth.to_bf16(x)
    _, _, xh2 = O.quant_act(xb[None, :], [16])
    assert np.array_equal(xh2[0], O.bf16_to_f64(xb))


def test_mlp_output_placement_of_the_quantizer():
    """The paper's placement (appendix "Activation quantization", "What is quantized"): the MLP output is
    quantized and dequantized before the residual add, the matmuls run at full precision, 16 bits and
    more leave it unchanged.  Checked against torch float32 library ops on the un-quantized MLP update."""
    import copy

    shape, W, kv, h = _layer_case(31)
    B = h.shape[0]
    r, p, bits = [1000, 500, 250][:B], [0, 250, 500][:B], [16, 12, 5][:B]
    out, tr = O.decode_layer(shape, W, copy.deepcopy(kv), h, r, p, bits, O.PLACE_MLP_OUTPUT)
    # the same layer with every width at 16 in the default placement gives the un-quantized MLP update z
    out16, tr16 = O.decode_layer(shape, W, copy.deepcopy(kv), h, r, p, [16] * B)
    z = out16 - tr16.h_mid
    assert np.allclose(tr.extra["z"], z, rtol=0, atol=1e-12)
    assert np.array_equal(tr.h_mid, tr16.h_mid)
    for i, b in enumerate(bits):
        got = out[i] - tr.h_mid[i]
        zi = tr.extra["z"][i]
        if b >= 16:
            assert np.array_equal(out[i], tr.h_mid[i] + zi)  # unchanged, not even rounded
            continue
        q_max = 2 ** (b - 1) - 1
        z32 = torch.from_numpy(zi).to(torch.float32)
        s = z32.abs().max() / q_max  # float32 division
        want = (torch.clamp(torch.round(z32 / s), -q_max, q_max).to(torch.float64) * s.to(torch.float64)).numpy()
        assert np.allclose(got, want, rtol=0, atol=1e-12), b
        assert np.all(np.abs(want - zi) <= 0.5 * float(s) * (1 + 1e-3))
        assert np.array_equal(tr.extra["z_codes"][i], np.round(want / float(s)).astype(np.int16))
    # the inputs of the projections are not quantized in this placement: codes all zero, scales 1
    assert not tr.codes1.any() and not tr.codes2.any() and np.all(tr.scales1 == 1) and np.all(tr.scales2 == 1)


def test_input_channel_gating_brute_force_ties_and_counts():
    """The paper's MLP pruning (appendix "Structured MLP activation pruning"): m = ceil(rho d) input channels of
    largest |x| survive.  Brute force over all subsets on a tiny row; ties to the lower index; the mask is 0/1."""
    import itertools
    from fractions import Fraction

    rng = np.random.default_rng(41)
    x = rng.standard_normal(9).astype(np.float32)
    for p in (0, 100, 250, 500, 667, 900, 1000):
        kept, masked = O.gate_input_channels(x, p)
        m = -((-(1000 - p) * 9) // 1000)  # ceil((1 - p) d)
        assert m == math.ceil(Fraction(1000 - p, 1000) * 9) and len(kept) == m
        best = max(itertools.combinations(range(9), m), key=lambda c: sum(abs(float(x[j])) for j in c)) if m else ()
        assert list(kept) == sorted(best)
        assert np.array_equal(masked[kept], x[kept]) and np.count_nonzero(masked) == m
    # equal magnitudes (either sign): the lower indices win
    t = np.array([1.0, -2.0, 2.0, -1.0, 2.0, 1.0], np.float32)
    assert list(O.gate_input_channels(t, 500)[0]) == [1, 2, 4]
    assert list(O.gate_input_channels(t, 667)[0]) == [1, 2]   # ceil(0.333 * 6) = 2
    assert list(O.gate_input_channels(t, 1000)[0]) == []


def test_layer_with_input_channel_gating_is_a_dense_mlp_on_the_masked_row():
    """PRUNE_MLP_INPUT: the MLP update equals a dense SwiGLU MLP (torch float64) on the masked, normalised row;
    the attention half of the layer is untouched; p = 0 reproduces the unpruned layer."""
    import copy

    shape, W, kv, h = _layer_case(43)
    B = h.shape[0]
    r, bits = [1000, 500, 250][:B], [16] * B
    p = [0, 500, 750][:B]
    out, tr = O.decode_layer(shape, W, copy.deepcopy(kv), h, r, p, bits, mlp_prune=O.PRUNE_MLP_INPUT)
    base, tr0 = O.decode_layer(shape, W, copy.deepcopy(kv), h, r, [0] * B, bits)
    assert np.array_equal(tr.h_mid, tr0.h_mid)  # attention input not pruned
    assert np.array_equal(out[0], base[0])      # p = 0 keeps every channel
    Wg, Wu, Wd = (torch.from_numpy(O.bf16_to_f64(m)) for m in (W.w_gate, W.w_up, W.w_down_t))
    d = shape.d_model
    for i in range(B):
        xn = torch.from_numpy(tr.xn2[i].astype(np.float64))
        m = -((-(1000 - p[i]) * d) // 1000)
        keep = torch.topk(xn.abs(), m).indices if m else torch.zeros(0, dtype=torch.long)
        assert sorted(keep.tolist()) == list(tr.extra["kept_inputs"][i])
        mask = torch.zeros(d, dtype=torch.float64)
        mask[keep] = 1.0
        xm = (xn * mask).to(torch.float32).to(torch.bfloat16).to(torch.float64)  # 16-bit passthrough of the masked row
        z = (torch.nn.functional.silu(Wg @ xm) * (Wu @ xm)) @ Wd
        assert np.allclose(out[i] - tr.h_mid[i], z.numpy(), rtol=0, atol=1e-12)
        assert len(tr.kept_channels[i]) == shape.d_ff  # no intermediate channel is dropped


def test_quantizer_mixed_bits_per_example():
    rng = np.random.default_rng(2)
    xb = synth.to_bf16(rng.standard_normal((3, 64)).astype(np.float32))
    codes, scales, xh = O.quant_act(xb, [4, 16, 8])
    for i, b in enumerate([4, 16, 8]):
        c, s, h = O.quant_act(xb[i:i + 1], [b])
        assert np.array_equal(c[0], codes[i]) and s[0] == scales[i] and np.array_equal(h[0], xh[i])
    for bad in (1, 17, 0):
        with pytest.raises(ValueError):
            O.quantize_per_token(np.ones(4, np.float32), bad)
    # widths over 8 bits carry int16 codes
    codes, scales, xh = O.quant_act(xb, [12, 16, 8])
    assert codes.dtype == np.int16 and np.abs(codes[0].astype(np.int64)).max() == 2047


# ------------------------------------------------------- rmsnorm / rope -----


def test_rmsnorm_matches_torch():
    rng = np.random.default_rng(3)
    h = rng.standard_normal(300) * 3
    g = 1 + 0.1 * rng.standard_normal(300)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(h), (300,), torch.from_numpy(g), 1e-5).numpy()
    assert np.allclose(O.rmsnorm(h, g, 1e-5), ref, rtol=1e-14, atol=0)


def test_rope_is_a_complex_rotation():
    rng = np.random.default_rng(4)
    hd, theta = 64, 500000.0
    v = rng.standard_normal((3, hd))
    for pos in [0, 1, 17, 4095, 32767]:
        z = v[:, : hd // 2] + 1j * v[:, hd // 2:]
        w = theta ** (-2.0 * np.arange(hd // 2) / hd)
        zr = z * np.exp(1j * pos * w)
        ref = np.concatenate([zr.real, zr.imag], axis=-1)
        assert np.allclose(O.rope_rotate(v, pos, theta), ref, rtol=0, atol=1e-12)
    assert np.array_equal(O.rope_rotate(v, 0, theta), v)
    assert np.array_equal(O.rope_rotate(v, 123, 0.0), v)


def test_rope_relative_position_property():
    rng = np.random.default_rng(5)
    q, k = rng.standard_normal(128), rng.standard_normal(128)
    a = O.rope_rotate(q, 1000, 10000.0) @ O.rope_rotate(k, 993, 10000.0)
    b = O.rope_rotate(q, 7, 10000.0) @ k
    assert abs(a - b) < 1e-9
    assert abs(np.linalg.norm(O.rope_rotate(q, 999, 10000.0)) - np.linalg.norm(q)) < 1e-12


# ------------------------------------------------------------ selection -----


def test_select_top_order_and_ties():
    s = np.array([1.0, 5.0, 5.0, 2.0, 5.0, 0.0])
    assert list(O.select_top(s, 2, np.array([], np.int64))) == [1, 2]  # ties -> lower index
    assert list(O.select_top(s, 3, np.array([5]))) == [1, 2, 5]  # forced counts toward k
    assert list(O.select_top(s, 1, np.array([5]))) == [5]
    assert list(O.select_top(s, 6, np.array([5]))) == [0, 1, 2, 3, 4, 5]


def _tiny_case(seed, T, G=2, hd=8, B=1, Hkv=1):
    rng = np.random.default_rng(seed)
    shape = O.Shape(d_model=16, n_q_heads=G * Hkv, n_kv_heads=Hkv, head_dim=hd, d_ff=12, page_size=4)
    n_pages = (T + 3) // 4
    k_pool = synth.to_bf16(rng.standard_normal((n_pages * B, Hkv, 4, hd)).astype(np.float32))
    v_pool = synth.to_bf16(rng.standard_normal((n_pages * B, Hkv, 4, hd)).astype(np.float32))
    table = np.arange(n_pages * B, dtype=np.int32).reshape(B, n_pages)
    kv = O.PagedKV(k_pool, v_pool, table, np.full(B, T, np.int32))
    q = rng.standard_normal((B, G * Hkv, hd))
    return shape, q, kv


def _dense_attention_torch(q, K, V, bias=None):
    """Library reference: torch SDPA in float64; q [G][hd], K,V [T][hd]."""
    qt = torch.from_numpy(q)[None, :, None, :]  # [1][G][1][hd]
    Kt = torch.from_numpy(K)[None, None].expand(1, q.shape[0], -1, -1)
    Vt = torch.from_numpy(V)[None, None].expand(1, q.shape[0], -1, -1)
    mask = None if bias is None else torch.from_numpy(bias)[None, None, None, :]
    return torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, attn_mask=mask)[0, :, 0, :].numpy()


@pytest.mark.parametrize("T,r", [(5, 400), (9, 334), (10, 500), (12, 250), (7, 1000), (6, 0)])
def test_token_selection_brute_force(T, r):
    """On tiny T the kept set is the unique subset of size k, containing the
    forced set, with the largest total score; the output is dense attention
    over a cache physically cut down to those rows."""
    shape, q, kv = _tiny_case(T * 1000 + r, T)
    out, kept, sigma = O.sparse_decode_attn(shape, q, kv, [r])
    kept, sigma = kept[0][0], sigma[0][0]
    k = min(T, max(1, math.ceil(Fraction(r, 1000) * T)))
    assert len(kept) == k and (T - 1) in kept
    K = O.cache_rows(kv.k_pool, kv.page_table[0], T, 0)
    V = O.cache_rows(kv.v_pool, kv.page_table[0], T, 0)
    score = (K @ q[0].T).sum(axis=1)
    assert np.allclose(score, sigma, rtol=1e-12)
    best, best_sum = None, -np.inf
    for sub in itertools.combinations(range(T - 1), k - 1):
        tot = score[list(sub)].sum()
        if tot > best_sum:
            best, best_sum = sub, tot
    assert sorted(best + (T - 1,)) == list(kept)
    ref = _dense_attention_torch(q[0], K[kept], V[kept])
    assert np.allclose(out[0], ref, rtol=1e-12, atol=1e-13)


def test_sparse_attention_equals_masked_dense():
    """The paper's own formulation: dropped keys get an additive -inf bias and
    the attention computation is otherwise unchanged."""
    shape, q, kv = _tiny_case(77, 23, G=4, hd=16)
    out, kept, _ = O.sparse_decode_attn(shape, q, kv, [300])
    K = O.cache_rows(kv.k_pool, kv.page_table[0], 23, 0)
    V = O.cache_rows(kv.v_pool, kv.page_table[0], 23, 0)
    bias = np.full(23, -np.inf)
    bias[kept[0][0]] = 0.0
    ref = _dense_attention_torch(q[0], K, V, bias)
    assert np.allclose(out[0], ref, rtol=1e-12, atol=1e-13)


def test_full_keep_rate_is_dense_gqa_attention():
    rng = np.random.default_rng(8)
    B, Hq, Hkv, hd, T = 3, 8, 2, 16, 37
    shape = O.Shape(d_model=32, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=hd, d_ff=8, page_size=8)
    n_pages = (T + 7) // 8
    perm = rng.permutation(B * n_pages).astype(np.int32).reshape(B, n_pages)  # shuffled pages
    k_pool = synth.to_bf16(rng.standard_normal((B * n_pages, Hkv, 8, hd)).astype(np.float32))
    v_pool = synth.to_bf16(rng.standard_normal((B * n_pages, Hkv, 8, hd)).astype(np.float32))
    lens = np.array([T, T - 5, 9], np.int32)
    kv = O.PagedKV(k_pool, v_pool, perm, lens)
    q = rng.standard_normal((B, Hq, hd))
    out, kept, _ = O.sparse_decode_attn(shape, q, kv, [1000, 1000, 1000])
    for i in range(B):
        Ti = int(lens[i])
        # assemble the contiguous cache by hand from the page table
        Kc = np.stack([np.concatenate([O.bf16_to_f64(k_pool[perm[i, p], h]) for p in range(n_pages)])[:Ti]
                       for h in range(Hkv)])
        Vc = np.stack([np.concatenate([O.bf16_to_f64(v_pool[perm[i, p], h]) for p in range(n_pages)])[:Ti]
                       for h in range(Hkv)])
        qt = torch.from_numpy(q[i])[None, :, None, :]
        Kt = torch.from_numpy(Kc)[None].repeat_interleave(Hq // Hkv, dim=1)
        Vt = torch.from_numpy(Vc)[None].repeat_interleave(Hq // Hkv, dim=1)
        ref = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)[0, :, 0, :].numpy()
        assert np.allclose(out[i], ref, rtol=1e-12, atol=1e-13)
        assert all(list(kk) == list(range(Ti)) for kk in kept[i])


def test_token_sets_nest_and_always_hold_newest():
    shape, q, kv = _tiny_case(9, 200, G=4, hd=16)
    prev = None
    for r in [0, 50, 125, 250, 500, 750, 1000]:
        _, kept, _ = O.sparse_decode_attn(shape, q, kv, [r])
        s = set(kept[0][0].tolist())
        assert 199 in s and len(s) == max(1, math.ceil(r * 200 / 1000))
        if prev is not None:
            assert prev <= s
        prev = s


def test_duplicate_keys_prefer_lower_index_and_sink_window():
    shape, q, kv = _tiny_case(10, 12)
    kv.k_pool[:] = kv.k_pool[0, 0, 0]  # every key identical: every score ties
    _, kept, _ = O.sparse_decode_attn(shape, q, kv, [500])
    assert list(kept[0][0]) == [0, 1, 2, 3, 4, 11]
    shape.n_sink, shape.n_window = 2, 3
    _, kept, _ = O.sparse_decode_attn(shape, q, kv, [500])
    assert list(kept[0][0]) == [0, 1, 2, 9, 10, 11]
    _, kept, _ = O.sparse_decode_attn(shape, q, kv, [100])  # budget 2 < 5 forced
    assert list(kept[0][0]) == [0, 1, 9, 10, 11]


# ---------------------------------------------------------------------------
# the paper's own token sparsity: Quest pages per query head
# ---------------------------------------------------------------------------
def _quest_golden():
    rows = []
    for line in open(os.path.join(GOLDEN, "quest_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        S, q, keys, r, scores, pages = [f.strip() for f in line.split(";")]
        rows.append((int(S), np.array(q.split(), float), np.array([k.split() for k in keys.split("|")], float), int(r),
                     np.array(scores.split(), float), np.array(pages.split(), int)))
    return rows


def test_quest_golden_scores_and_pages():
    rows = _quest_golden()
    assert len(rows) >= 9
    for S, q, K, r, scores, pages in rows:
        T = K.shape[0]
        mp, mm = O.quest_page_extrema(K, S)
        assert np.array_equal(O.quest_page_scores(q, mp, mm), scores)
        forced = np.unique(O.forced_keep_set(T, 0, 1) // S)
        n = O.quest_kept_page_count(r, T, S, len(forced))
        assert n == len(pages)
        _, kept, sc = O.quest_attention_one_group(q[None], K, np.zeros_like(K), S, n, forced)
        assert np.array_equal(kept[0], pages) and np.array_equal(sc[0], scores)


@pytest.mark.parametrize("S", [1, 4, 16])
def test_quest_score_bounds_every_key_of_the_page(S):
    rng = np.random.default_rng(S)
    K = rng.normal(size=(131, 16))
    for q in rng.normal(size=(5, 16)):
        mp, mm = O.quest_page_extrema(K, S)
        sc = O.quest_page_scores(q, mp, mm)
        dots = K @ q
        for pg in range(len(sc)):
            top = dots[pg * S:(pg + 1) * S].max()
            assert sc[pg] >= top - 1e-12
            if S == 1:
                assert abs(sc[pg] - top) < 1e-12  # a page of one key: the bound is the dot product
        # the bound is the sum over dimensions of max(q_d min_d, q_d max_d): the largest any point of the box can give
        lo = np.stack([K[pg * S:(pg + 1) * S].min(axis=0) for pg in range(len(sc))])
        hi = np.stack([K[pg * S:(pg + 1) * S].max(axis=0) for pg in range(len(sc))])
        assert np.allclose(sc, np.maximum(lo * q, hi * q).sum(axis=1), rtol=0, atol=1e-12)


def test_quest_kept_page_count_closed_form():
    for T in (1, 5, 16, 17, 100, 1000):
        for S in (1, 4, 8, 16):
            for r in (0, 1, 125, 333, 500, 999, 1000):
                b = min(T, max(0, math.ceil(Fraction(r, 1000) * T)))
                want = min(-(-T // S), max(-(-b // S), 1))
                assert O.quest_kept_page_count(r, T, S, 1) == want
    with pytest.raises(ValueError):
        O.quest_kept_page_count(1001, 10, 4, 1)


@pytest.mark.parametrize("S,r", [(1, 300), (4, 250), (8, 600), (16, 125)])
def test_quest_attention_is_masked_dense_attention_per_head(S, r):
    """Brute force: per head, rank the pages by the bound with a stable sort, expand to a token mask, and run
    a dense softmax with an additive -inf bias in torch."""
    rng = np.random.default_rng(100 + S)
    T, hd, G = 77, 8, 3
    K, V, qg = rng.normal(size=(T, hd)), rng.normal(size=(T, hd)), rng.normal(size=(G, hd))
    P = -(-T // S)
    last = (T - 1) // S
    n = O.quest_kept_page_count(r, T, S, 1)
    out, kept, sc = O.quest_attention_one_group(qg, K, V, S, n, np.array([last]))
    for h in range(G):
        lo = np.stack([K[pg * S:(pg + 1) * S].min(axis=0) for pg in range(P)])
        hi = np.stack([K[pg * S:(pg + 1) * S].max(axis=0) for pg in range(P)])
        bound = np.maximum(lo * qg[h], hi * qg[h]).sum(axis=1)
        others = [pg for pg in sorted(range(P), key=lambda pg: (-bound[pg], pg)) if pg != last]
        want = sorted([last] + others[: n - 1])
        assert list(kept[h]) == want
        bias = torch.full((T,), float("-inf"), dtype=torch.float64)
        for pg in want:
            bias[pg * S:(pg + 1) * S] = 0.0
        w = torch.softmax(torch.from_numpy(K @ qg[h] / math.sqrt(hd)) + bias, dim=0)
        assert np.allclose(out[h], (w[:, None] * torch.from_numpy(V)).sum(0).numpy(), rtol=0, atol=1e-12)


def _small_paged_case(seed):
    rng = np.random.default_rng(seed)
    B, Hq, Hkv, hd, T = 3, 8, 2, 16, 53
    shape = O.Shape(d_model=32, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=hd, d_ff=8, page_size=8)
    n_pages = (T + 7) // 8
    perm = rng.permutation(B * n_pages).astype(np.int32).reshape(B, n_pages)  # shuffled pages
    k_pool = synth.to_bf16(rng.standard_normal((B * n_pages, Hkv, 8, hd)).astype(np.float32))
    v_pool = synth.to_bf16(rng.standard_normal((B * n_pages, Hkv, 8, hd)).astype(np.float32))
    kv = O.PagedKV(k_pool, v_pool, perm, np.array([T, T - 5, 9], np.int32))
    return shape, kv, rng.standard_normal((B, Hq, hd)), B


def test_quest_full_keep_rate_is_dense_and_pages_nest():
    shape, kv, q, B = _small_paged_case(3)
    dense, _, _ = O.sparse_decode_attn(shape, q, kv, [1000] * B)
    for S in (4, 16):
        out, kept, _ = O.quest_decode_attn(shape, q, kv, [1000] * B, S)
        assert np.allclose(out, dense, rtol=0, atol=1e-12)
        prev = None
        for r in (0, 125, 250, 500, 1000):
            _, kept, _ = O.quest_decode_attn(shape, q, kv, [r] * B, S)
            for i in range(B):
                last = (int(kv.seq_lens[i]) - 1) // S
                assert all(last in set(pg) for pg in kept[i])
                assert len(kept[i]) == shape.n_q_heads
            if prev is not None:
                assert all(set(a) <= set(b) for i in range(B) for a, b in zip(prev[i], kept[i]))
            prev = kept


def test_quest_heads_select_independently():
    """Selection is per query head: changing one head's query changes only that head's pages and output."""
    shape, kv, q, B = _small_paged_case(4)
    out0, kept0, _ = O.quest_decode_attn(shape, q, kv, [250] * B, 8)
    q2 = q.copy()
    q2[:, 1] = -q2[:, 1]
    out1, kept1, _ = O.quest_decode_attn(shape, q2, kv, [250] * B, 8)
    for h in range(shape.n_q_heads):
        same = all(np.array_equal(kept0[i][h], kept1[i][h]) for i in range(B))
        if h != 1:
            assert same and np.array_equal(out0[:, h], out1[:, h])
    assert not np.array_equal(out0[:, 1], out1[:, 1])


def test_attention_output_is_a_convex_combination():
    shape, q, kv = _tiny_case(11, 40, G=2, hd=8)
    out, kept, _ = O.sparse_decode_attn(shape, q, kv, [250])
    V = O.cache_rows(kv.v_pool, kv.page_table[0], 40, 0)[kept[0][0]]
    assert np.all(out[0] <= V.max(axis=0) + 1e-12) and np.all(out[0] >= V.min(axis=0) - 1e-12)


def test_batch_rows_are_independent():
    shape, q, kv = _tiny_case(12, 30, B=3, Hkv=2)
    r = [250, 1000, 500]
    out, kept, _ = O.sparse_decode_attn(shape, q, kv, r)
    for i in range(3):
        kv1 = O.PagedKV(kv.k_pool, kv.v_pool, kv.page_table[i:i + 1], kv.seq_lens[i:i + 1])
        o1, k1, _ = O.sparse_decode_attn(shape, q[i:i + 1], kv1, r[i:i + 1])
        assert np.array_equal(o1[0], out[i])
        assert all(np.array_equal(a, b) for a, b in zip(k1[0], kept[i]))


# ------------------------------------------------------------------ MLP -----


def _mlp_case(seed, B=3, d=24, ff=40):
    rng = np.random.default_rng(seed)
    w = lambda *s: synth.to_bf16((rng.standard_normal(s) * 0.3).astype(np.float32))
    return rng.standard_normal((B, d)), w(ff, d), w(ff, d), w(ff, d)


def test_dense_mlp_matches_torch():
    x, wg, wu, wd = _mlp_case(20)
    out, kept, t = O.pruned_swiglu_mlp(x, wg, wu, wd, [0, 0, 0])
    xt = torch.from_numpy(x)
    ref = (torch.nn.functional.silu(xt @ t64(wg).T) * (xt @ t64(wu).T)) @ t64(wd)
    assert np.allclose(out, ref.numpy(), rtol=1e-12, atol=1e-13)
    assert all(list(k) == list(range(40)) for k in kept)


@pytest.mark.parametrize("p", [250, 500, 600, 900, 1000])
def test_pruned_mlp_brute_force_and_masked_dense(p):
    x, wg, wu, wd = _mlp_case(21 + p, B=2, d=10, ff=11)
    out, kept, t = O.pruned_swiglu_mlp(x, wg, wu, wd, [p, p])
    xt = torch.from_numpy(x)
    t_ref = (torch.nn.functional.silu(xt @ t64(wg).T) * (xt @ t64(wu).T)).numpy()
    assert np.allclose(t, t_ref, rtol=1e-12, atol=1e-14)
    m = math.ceil(Fraction(1000 - p, 1000) * 11)
    for i in range(2):
        assert len(kept[i]) == m
        best = max(itertools.combinations(range(11), m), key=lambda s: np.abs(t_ref[i, list(s)]).sum()) if m else ()
        assert sorted(best) == list(kept[i])
        masked = np.zeros(11)
        masked[list(best)] = t_ref[i, list(best)]
        ref = masked @ O.bf16_to_f64(wd)  # dense down-projection with the dropped channels zeroed
        assert np.allclose(out[i], ref, rtol=1e-12, atol=1e-14)
    if p == 1000:
        assert not out.any()


def test_channel_sets_nest_and_tie_break():
    x, wg, wu, wd = _mlp_case(30, B=1, d=16, ff=64)
    prev = None
    for p in [1000, 750, 500, 250, 0]:
        _, kept, _ = O.pruned_swiglu_mlp(x, wg, wu, wd, [p])
        s = set(kept[0].tolist())
        if prev is not None:
            assert prev <= s
        prev = s
    wg[:] = wg[0]
    wu[:] = wu[0]  # all channels identical -> all |t| tie -> lowest indices kept
    _, kept, _ = O.pruned_swiglu_mlp(x, wg, wu, wd, [750])
    assert list(kept[0]) == list(range(16))


# ---------------------------------------------------------------- layer -----


def _layer_case(seed, B=3, T=21, theta=10000.0):
    cfg = dict(d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48)
    rng = np.random.default_rng(seed)
    shape = O.Shape(page_size=4, rope_theta=theta, **cfg)
    w = lambda *s: synth.to_bf16((rng.standard_normal(s) * 0.2).astype(np.float32))
    d, hq, hkv, hd, ff = 32, 4, 2, 8, 48
    W = O.LayerWeights(w((hq + 2 * hkv) * hd, d), w(d, hq * hd), w(ff, d), w(ff, d), w(ff, d),
                       synth.to_bf16((1 + 0.1 * rng.standard_normal(d)).astype(np.float32)),
                       synth.to_bf16((1 + 0.1 * rng.standard_normal(d)).astype(np.float32)))
    lens = np.array([T, T - 4, 5][:B], np.int32)
    n_pages = (T + 3) // 4
    table = rng.permutation(B * n_pages).astype(np.int32).reshape(B, n_pages)
    kv = O.PagedKV(synth.to_bf16(rng.standard_normal((B * n_pages, hkv, 4, hd)).astype(np.float32)),
                   synth.to_bf16(rng.standard_normal((B * n_pages, hkv, 4, hd)).astype(np.float32)), table, lens)
    h = O.bf16_to_f64(synth.to_bf16(rng.standard_normal((B, d)).astype(np.float32)))
    return shape, W, kv, h


def _dense_layer_torch(shape, W, kv, h):
    """Textbook Llama decoder layer for one new token per sequence, written
    with torch library ops in float64; activations pass through bf16 where a
    bf16 pipeline would carry them (b = 16)."""
    B, d = h.shape
    Hq, Hkv, hd, P = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.page_size
    F = torch.nn.functional
    ht = torch.from_numpy(h)

    def carried(x):  # float64 -> float32 -> bf16 -> float64
        return x.to(torch.float32).to(torch.bfloat16).to(torch.float64)

    def rot(x, pos):  # x [heads][hd]
        if shape.rope_theta == 0:
            return x
        inv = shape.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
        ang = torch.cat([pos * inv, pos * inv])
        x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
        return x * torch.cos(ang) + torch.cat([-x2, x1], dim=-1) * torch.sin(ang)

    x = carried(F.rms_norm(ht, (d,), t64(W.gamma1), shape.rms_eps))
    qkv = F.linear(x, t64(W.w_qkv))
    out = torch.zeros(B, Hq * hd, dtype=torch.float64)
    k_pool, v_pool = kv.k_pool.copy(), kv.v_pool.copy()
    for i in range(B):
        T = int(kv.seq_lens[i])
        q = rot(qkv[i, : Hq * hd].view(Hq, hd), T - 1)
        k = rot(qkv[i, Hq * hd:(Hq + Hkv) * hd].view(Hkv, hd), T - 1)
        v = qkv[i, (Hq + Hkv) * hd:].view(Hkv, hd)
        pg, slot = int(kv.page_table[i, (T - 1) // P]), (T - 1) % P
        k_pool[pg, :, slot] = k.to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        v_pool[pg, :, slot] = v.to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        pages = [int(kv.page_table[i, p]) for p in range((T + P - 1) // P)]
        Kc = t64(np.concatenate([k_pool[p] for p in pages], axis=1)[:, :T])  # [Hkv][T][hd]
        Vc = t64(np.concatenate([v_pool[p] for p in pages], axis=1)[:, :T])
        o = F.scaled_dot_product_attention(q[None, :, None, :], Kc[None].repeat_interleave(Hq // Hkv, 1),
                                           Vc[None].repeat_interleave(Hq // Hkv, 1))
        out[i] = o.reshape(-1)
    h_mid = ht + F.linear(out, t64(W.w_o))
    x2 = carried(F.rms_norm(h_mid, (d,), t64(W.gamma2), shape.rms_eps))
    mlp = (F.silu(F.linear(x2, t64(W.w_gate))) * F.linear(x2, t64(W.w_up))) @ t64(W.w_down_t)
    return (h_mid + mlp).numpy(), k_pool, v_pool


@pytest.mark.parametrize("theta", [0.0, 10000.0])
def test_dense_action_reproduces_textbook_layer(theta):
    """r = 1, p = 0, b = 16 recovers the dense path."""
    shape, W, kv, h = _layer_case(40, theta=theta)
    ref, k_ref, v_ref = _dense_layer_torch(shape, W, kv, h)
    out, tr = O.decode_layer(shape, W, kv, h, [1000] * 3, [0] * 3, [16] * 3)
    assert np.allclose(out, ref, rtol=1e-11, atol=1e-12)
    # appended rows match up to the double rounding (float64 -> float32 -> bf16) of the torch path
    assert np.max(np.abs(kv.k_pool.astype(np.int64) - k_ref.astype(np.int64))) <= 1
    assert np.max(np.abs(kv.v_pool.astype(np.int64) - v_ref.astype(np.int64))) <= 1
    assert np.mean(kv.k_pool != k_ref) < 1e-3


def test_layer_appends_at_the_newest_position_only():
    shape, W, kv, h = _layer_case(41)
    k0, v0 = kv.k_pool.copy(), kv.v_pool.copy()
    O.decode_layer(shape, W, kv, h, [500] * 3, [250] * 3, [8] * 3)
    changed = np.argwhere((kv.k_pool != k0).any(axis=(1, 3)))  # (page, slot)
    want = sorted((int(kv.page_table[i, (int(T) - 1) // 4]), (int(T) - 1) % 4) for i, T in enumerate(kv.seq_lens))
    assert sorted(set(map(tuple, changed.tolist()))) == want
    assert sorted(set(map(tuple, np.argwhere((kv.v_pool != v0).any(axis=(1, 3))).tolist()))) == want


def test_layer_composes_its_parts_with_mixed_actions():
    """Each action axis acts where the definitions say: recompute the layer
    from the stand-alone pieces and the trace."""
    shape, W, kv, h = _layer_case(42)
    r, p, b = [250, 1000, 500], [500, 0, 250], [4, 16, 8]
    kv_before = O.PagedKV(kv.k_pool.copy(), kv.v_pool.copy(), kv.page_table, kv.seq_lens)
    out, tr = O.decode_layer(shape, W, kv, h, r, p, b)
    for i in range(3):
        # quantized attention input
        xn = O.rmsnorm(h[i], O.bf16_to_f64(W.gamma1), shape.rms_eps).astype(np.float32)
        c, s, xh = O.quantize_per_token(xn, b[i])
        assert np.array_equal(c, tr.codes1[i]) and s == tr.scales1[i]
        qkv = O.bf16_to_f64(W.w_qkv) @ xh
        T = int(kv.seq_lens[i])
        q = O.rope_rotate(qkv[: 32].reshape(4, 8), T - 1, shape.rope_theta)
        assert np.allclose(q, tr.q_rot[i], rtol=1e-13, atol=1e-15)
        assert len(tr.kept_tokens[i][0]) == max(1, math.ceil(r[i] * T / 1000))
        assert len(tr.kept_channels[i]) == math.ceil((1000 - p[i]) * 48 / 1000)
    # attention reads the cache AFTER the append
    attn, kept, _ = O.sparse_decode_attn(shape, tr.q_rot, kv, r)
    assert np.array_equal(attn, tr.attn_out)
    attn_stale, _, _ = O.sparse_decode_attn(shape, tr.q_rot, kv_before, r)
    assert not np.allclose(attn_stale, attn)
    h_mid = h + attn.reshape(3, -1) @ O.bf16_to_f64(W.w_o).T
    assert np.allclose(h_mid, tr.h_mid, rtol=1e-13)
    _, _, _, xh2 = O.norm_and_quantize(h_mid, W.gamma2, shape.rms_eps, b)
    mlp, _, _ = O.pruned_swiglu_mlp(xh2, W.w_gate, W.w_up, W.w_down_t, p)
    assert np.allclose(out, h_mid + mlp, rtol=1e-13)


def test_decode_step_stacks_layers_with_one_action():
    shape, W, kv, h = _layer_case(43)
    shape2, W2, kv2, _ = _layer_case(44)
    hb = synth.to_bf16(h.astype(np.float32))
    r, p, b = [500, 250, 1000], [250, 500, 0], [8, 4, 16]
    kva = [O.PagedKV(k.k_pool.copy(), k.v_pool.copy(), k.page_table, k.seq_lens) for k in (kv, kv2)]
    out, traces = O.decode_step(shape, [W, W2], kva, hb, r, p, b)
    h1, _ = O.decode_layer(shape, W, kv, O.bf16_to_f64(hb), r, p, b)
    h2, _ = O.decode_layer(shape, W2, kv2, h1, r, p, b)
    assert np.array_equal(out, h2) and len(traces) == 2


# ------------------------------------------------------------- workloads ----


def test_synth_is_seeded_and_shaped():
    cfg = synth.WORKLOADS["tiny"]
    a, b = synth.make_layer_weights(cfg, 0), synth.make_layer_weights(cfg, 0)
    assert np.array_equal(a.w_qkv, b.w_qkv) and a.w_qkv.shape == (512, 256) and a.w_down_t.shape == (1024, 256)
    assert not np.array_equal(a.w_gate, a.w_up)
    w = O.bf16_to_f64(a.w_gate)
    assert abs(w.std() - 0.02) < 1e-3 and abs(w.mean()) < 1e-3
    lens = synth.make_contexts(synth.WORKLOADS["ragged_serving"], 0)
    assert lens.min() >= 256 and lens.max() <= 32768 and len(lens) == 128
    tab, n = synth.make_page_table(np.array([130, 64, 1]), True, 0)
    ids = tab[tab >= 0]
    assert n == 5 and sorted(ids.tolist()) == list(range(5)) and tab.shape == (3, 3)
    r, p, bb = synth.draw_actions(synth.WORKLOADS["llama1b_layer"], 0)
    assert set(r) <= {125, 250, 500, 1000} and set(p) <= {0, 250, 500, 750} and set(bb) <= {4, 8, 16}
    for tgt in [125, 250, 375, 500, 1000]:
        r, p, bb = synth.budget_mix_actions(synth.WORKLOADS["llama1b_step"], tgt, 0)
        assert abs(np.mean(r * (1000 - p) / 1000.0) - tgt) <= 1000 / 32
    x = np.random.default_rng(0).standard_normal(5000).astype(np.float32)
    assert np.array_equal(synth.to_bf16(x), torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


# --------------------------------------------------------------- checker ----


def test_checker_near_tie_rule_and_output_bounds():
    from oracle import checker

    score = np.array([5.0, 4.0, 3.0000001, 3.0, 1.0])
    ok = checker.compare_index_set(score, np.array([0, 1, 2]), np.array([0, 1, 2]))
    assert ok.exact == 1 and ok.ok()
    tie = checker.compare_index_set(score, np.array([0, 1, 2]), np.array([0, 1, 3]))
    assert tie.ok() and tie.near_tie_indices == 2 and tie.exact == 0
    bad = checker.compare_index_set(score, np.array([0, 1, 2]), np.array([0, 1, 4]))
    assert not bad.ok() and bad.failed_indices >= 1
    assert not checker.compare_index_set(score, np.array([0, 1, 2]), np.array([0, 1])).ok()
    assert not checker.compare_index_set(score, np.array([0, 1, 2]), np.array([0, 1, 1])).ok()
    # forced indices are never excused
    f = checker.compare_index_set(score, np.array([0, 1, 4]), np.array([0, 1, 3]), forced=np.array([4]))
    assert not f.ok()
    o = np.array([1.0, -7.9, 9.0, 20.0])
    assert checker.outputs_ok(o, o + np.array([0.019, 0.019, 0.039, 0.079]))
    assert not checker.outputs_ok(o, o + np.array([0.021, 0, 0, 0]))
    assert not checker.outputs_ok(o, o + np.array([0, 0, 0.041, 0]))
    m, rel = checker.output_errors(np.ones(4), np.ones(4) * 1.02)
    assert abs(m - 0.02) < 1e-12 and abs(rel - 0.02) < 1e-12


# ---------------------------------------------------------- KV refresh ------


def _refresh_case(seed, n, L=2, theta=10000.0):
    """L small layers, three paged sequences whose last n tokens are to be refreshed, and the span's inputs."""
    rng = np.random.default_rng(seed)
    shape, _, _, _ = _layer_case(seed, theta=theta)
    d, hq, hkv, hd, ff = 32, 4, 2, 8, 48
    w = lambda *s: synth.to_bf16((rng.standard_normal(s) * 0.2).astype(np.float32))
    layers = [O.LayerWeights(w((hq + 2 * hkv) * hd, d), w(d, hq * hd), w(ff, d), w(ff, d), w(ff, d),
                             synth.to_bf16((1 + 0.1 * rng.standard_normal(d)).astype(np.float32)),
                             synth.to_bf16((1 + 0.1 * rng.standard_normal(d)).astype(np.float32))) for _ in range(L)]
    lens = np.array([21, 17, n], np.int32)  # the last sequence is nothing but the span
    n_pages = 6
    table = rng.permutation(3 * n_pages).astype(np.int32).reshape(3, n_pages)
    pools = [(synth.to_bf16(rng.standard_normal((3 * n_pages, hkv, 4, hd)).astype(np.float32)),
              synth.to_bf16(rng.standard_normal((3 * n_pages, hkv, 4, hd)).astype(np.float32))) for _ in range(L)]
    h_span = synth.to_bf16(rng.standard_normal((3, n, d)).astype(np.float32))
    return shape, layers, pools, table, lens, h_span


def _causal_prefill_layer_torch(shape, W, k_pool, v_pool, table, lens, h):
    """Textbook causal prefill of one Llama layer over the last n tokens of each sequence, with torch library ops
    in float64: all n keys and values are written first, then one masked attention call per sequence.
    h float64 [B][n][d]; returns the outputs and the new pools."""
    B, n, d = h.shape
    Hq, Hkv, hd, P = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.page_size
    F = torch.nn.functional
    carried = lambda x: x.to(torch.float32).to(torch.bfloat16).to(torch.float64)
    as_u16 = lambda x: x.to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)

    def rot(x, pos):  # x [n][heads][hd], pos [n]
        if shape.rope_theta == 0:
            return x
        inv = shape.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
        ang = torch.cat([pos[:, None] * inv, pos[:, None] * inv], dim=-1)[:, None, :]
        x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
        return x * torch.cos(ang) + torch.cat([-x2, x1], dim=-1) * torch.sin(ang)

    ht = torch.from_numpy(h)
    x = carried(F.rms_norm(ht, (d,), t64(W.gamma1), shape.rms_eps))
    qkv = F.linear(x, t64(W.w_qkv))  # [B][n][...]
    k_pool, v_pool = k_pool.copy(), v_pool.copy()
    attn = torch.zeros(B, n, Hq * hd, dtype=torch.float64)
    for i in range(B):
        T = int(lens[i])
        pos = torch.arange(T - n, T, dtype=torch.float64)
        q = rot(qkv[i, :, : Hq * hd].view(n, Hq, hd), pos)
        k = rot(qkv[i, :, Hq * hd:(Hq + Hkv) * hd].view(n, Hkv, hd), pos)
        v = qkv[i, :, (Hq + Hkv) * hd:].view(n, Hkv, hd)
        for j in range(n):
            t = T - n + j
            k_pool[int(table[i, t // P]), :, t % P] = as_u16(k[j])
            v_pool[int(table[i, t // P]), :, t % P] = as_u16(v[j])
        pages = [int(table[i, p]) for p in range((T + P - 1) // P)]
        Kc = t64(np.concatenate([k_pool[p] for p in pages], axis=1)[:, :T])  # [Hkv][T][hd]
        Vc = t64(np.concatenate([v_pool[p] for p in pages], axis=1)[:, :T])
        mask = torch.arange(T)[None, :] <= (T - n + torch.arange(n))[:, None]  # query j sees keys up to its own
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], Kc[None].repeat_interleave(Hq // Hkv, 1),
                                           Vc[None].repeat_interleave(Hq // Hkv, 1), attn_mask=mask)
        attn[i] = o[0].transpose(0, 1).reshape(n, Hq * hd)
    h_mid = ht + F.linear(attn, t64(W.w_o))
    x2 = carried(F.rms_norm(h_mid, (d,), t64(W.gamma2), shape.rms_eps))
    mlp = (F.silu(F.linear(x2, t64(W.w_gate))) * F.linear(x2, t64(W.w_up))) @ t64(W.w_down_t)
    return (h_mid + mlp).numpy(), k_pool, v_pool


@pytest.mark.parametrize("n,theta", [(1, 10000.0), (5, 10000.0), (8, 0.0)])
def test_kv_refresh_is_a_textbook_causal_prefill(n, theta):
    shape, layers, pools, table, lens, h_span = _refresh_case(50 + n, n, theta=theta)
    kvs = [O.PagedKV(k.copy(), v.copy(), table, lens.copy()) for k, v in pools]
    out = O.kv_refresh(shape, layers, kvs, h_span)
    h = O.bf16_to_f64(h_span)
    for l, W in enumerate(layers):
        h, k_ref, v_ref = _causal_prefill_layer_torch(shape, W, pools[l][0], pools[l][1], table, lens, h)
        # cache entries agree up to the double rounding of the torch path (float64 -> float32 -> bf16)
        assert np.max(np.abs(kvs[l].k_pool.astype(np.int64) - k_ref.astype(np.int64))) <= 1
        assert np.max(np.abs(kvs[l].v_pool.astype(np.int64) - v_ref.astype(np.int64))) <= 1
        assert np.mean(kvs[l].k_pool != k_ref) < 2e-3
    assert np.allclose(out, h, rtol=1e-9, atol=1e-9)
    assert all(np.array_equal(kv.seq_lens, lens) for kv in kvs)


def test_kv_refresh_restores_the_dense_cache_after_polluted_steps():
    """The paper's purpose of the refresh: n decode steps under aggressive actions leave cache entries that
    differ from the dense ones; the refresh over the same n tokens rebuilds exactly what n dense steps write."""
    n = 4
    shape, layers, pools, table, lens, h_span = _refresh_case(60, n)
    B = 3
    dense_kvs = [O.PagedKV(k.copy(), v.copy(), table, lens.copy()) for k, v in pools]
    dirty_kvs = [O.PagedKV(k.copy(), v.copy(), table, lens.copy()) for k, v in pools]
    dense_out = np.zeros((B, n, 32))
    for i in range(n):  # token-by-token decode, both ways
        for kv in dense_kvs + dirty_kvs:
            kv.seq_lens = (lens - n + 1 + i).astype(np.int32)
        dense_out[:, i], _ = O.decode_step(shape, layers, dense_kvs, h_span[:, i], [1000] * B, [0] * B, [16] * B)
        O.decode_step(shape, layers, dirty_kvs, h_span[:, i], [250] * B, [500] * B, [4] * B)
    for kv in dense_kvs + dirty_kvs:
        kv.seq_lens = lens.copy()
    assert any(not np.array_equal(a.k_pool, b.k_pool) for a, b in zip(dense_kvs, dirty_kvs))
    out = O.kv_refresh(shape, layers, dirty_kvs, h_span)
    for a, b in zip(dense_kvs, dirty_kvs):
        assert np.array_equal(a.k_pool, b.k_pool) and np.array_equal(a.v_pool, b.v_pool)
    assert np.array_equal(out, dense_out)
    # a second refresh changes nothing
    before = [(kv.k_pool.copy(), kv.v_pool.copy()) for kv in dirty_kvs]
    out2 = O.kv_refresh(shape, layers, dirty_kvs, h_span)
    assert np.array_equal(out, out2)
    assert all(np.array_equal(kv.k_pool, k) and np.array_equal(kv.v_pool, v) for kv, (k, v) in zip(dirty_kvs, before))


def test_kv_refresh_touches_the_span_only():
    n = 5
    shape, layers, pools, table, lens, h_span = _refresh_case(61, n)
    kvs = [O.PagedKV(k.copy(), v.copy(), table, lens.copy()) for k, v in pools]
    O.kv_refresh(shape, layers, kvs, h_span)
    want = sorted((int(table[i, t // 4]), t % 4) for i, T in enumerate(lens) for t in range(int(T) - n, int(T)))
    for l, kv in enumerate(kvs):
        for new, old in ((kv.k_pool, pools[l][0]), (kv.v_pool, pools[l][1])):
            changed = sorted(set(map(tuple, np.argwhere((new != old).any(axis=(1, 3))).tolist())))
            assert changed == want
