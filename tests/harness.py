"""Glue for the GPU parity tests: moves seeded NumPy inputs into torch device
tensors (torch is used for device memory only), calls the C ABI through the
binding, brings results back as NumPy, and compares them with the oracle."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from oracle import checker
from oracle import sol_oracle as O
from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth

DEV = "cuda:0"


def dev_bf16(u16: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(u16).view(np.int16)).to(DEV).view(torch.bfloat16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(np.asarray(a, np.int32))).to(DEV)


def host_u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def make_shapes(cfg: dict, n_sink=0, n_window=1, quant_placement=0, mlp_prune=0, token_select=0, quest_page_size=0):
    kw = dict(d_model=cfg["d_model"], n_q_heads=cfg["n_q_heads"], n_kv_heads=cfg["n_kv_heads"],
              head_dim=cfg["head_dim"], d_ff=cfg["d_ff"], page_size=64, rms_eps=synth.RMS_EPS,
              rope_theta=cfg.get("rope_theta", 0.0), n_sink=n_sink, n_window=n_window)
    return sol.make_shape(quant_placement=quant_placement, mlp_prune=mlp_prune, token_select=token_select,
                          quest_page_size=quest_page_size, **kw), O.Shape(**kw)


class Workspace:
    def __init__(self, shape, max_batch: int, max_pages: int):
        self.bytes = sol.workspace_bytes(shape, max_batch, max_pages)
        assert self.bytes > 0, "unsupported shape"
        self.buf = torch.empty(self.bytes, dtype=torch.uint8, device=DEV)
        sol.workspace_init(self.buf, self.bytes)
        torch.cuda.synchronize()

    def status(self) -> List[int]:
        return sol.read_device_status(self.buf)


@dataclass
class DeviceKV:
    k_pool: torch.Tensor
    v_pool: torch.Tensor
    page_table: torch.Tensor
    seq_lens: torch.Tensor
    max_pages: int
    num_pages: int
    quest_meta: Optional[torch.Tensor] = None

    def struct(self):
        return sol.make_kv(self.k_pool, self.v_pool, self.page_table, self.seq_lens, self.max_pages, self.num_pages,
                           self.quest_meta)

    def build_quest_meta(self, shape, B: int):
        """Allocates the page extrema for a shape in Quest mode and fills them from the cache."""
        n = sol.quest_meta_bytes(shape, self.num_pages)
        assert n > 0
        self.quest_meta = torch.zeros(n // 2, dtype=torch.bfloat16, device=DEV)
        sol.quest_build_meta(shape, self.struct(), B)
        torch.cuda.synchronize()

    def to_oracle(self) -> O.PagedKV:
        return O.PagedKV(host_u16(self.k_pool), host_u16(self.v_pool), self.page_table.cpu().numpy(),
                         self.seq_lens.cpu().numpy())


def device_kv(k_pool: np.ndarray, v_pool: np.ndarray, page_table: np.ndarray, seq_lens: np.ndarray) -> DeviceKV:
    table = np.where(page_table < 0, 0, page_table).astype(np.int32)
    return DeviceKV(dev_bf16(k_pool), dev_bf16(v_pool), dev_i32(table), dev_i32(seq_lens), page_table.shape[1],
                    k_pool.shape[0])


def make_case_kv(cfg: dict, seq_lens: np.ndarray, seed=0, layer=0, shuffle=None, spare_tokens=0):
    shuffle = cfg.get("shuffle_pages", True) if shuffle is None else shuffle
    table, n_pages = synth.make_page_table(seq_lens, shuffle, seed, spare_tokens)
    k_pool, v_pool = synth.make_kv_pool(cfg, n_pages, seed, layer)
    return k_pool, v_pool, table


def pack_layer(shape, plain: dict) -> dict:
    """Packs the four matrices of a layer (device bf16 tensors, row-major) with sol_pack_weights; returns the
    packed device buffers and the gains.  The row-major tensors can be dropped afterwards."""
    out = {"gamma1": plain["gamma1"], "gamma2": plain["gamma2"]}
    for name, kind, a, b in (("w_qkv", sol.W_QKV, "w_qkv", None), ("w_o", sol.W_O, "w_o", None),
                             ("w_gate_up", sol.W_GATE_UP, "w_gate", "w_up"), ("w_down", sol.W_DOWN, "w_down_t", None)):
        n = sol.packed_weight_bytes(shape, kind)
        assert n > 0, (name, "unsupported shape")
        buf = torch.empty(n, dtype=torch.uint8, device=plain[a].device)
        sol.pack_weights(shape, kind, plain[a], plain[b] if b else None, buf, n)
        out[name] = buf
    torch.cuda.synchronize()
    return out


@dataclass
class DeviceWeights:
    tensors: dict  # packed matrices + gains

    def struct(self):
        t = self.tensors
        return sol.make_weights(t["w_qkv"], t["w_o"], t["w_gate_up"], t["w_down"], t["gamma1"], t["gamma2"])


def device_weights(w: synth.LayerTensors, shape) -> DeviceWeights:
    """Uploads a layer's row-major weights and packs them for the library (shape: a sol shape of the layer)."""
    plain = {n: dev_bf16(getattr(w, n)) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down_t", "gamma1", "gamma2")}
    return DeviceWeights(pack_layer(shape, plain))


def oracle_weights(w: synth.LayerTensors) -> O.LayerWeights:
    return O.LayerWeights(w.w_qkv, w.w_o, w.w_gate, w.w_up, w.w_down_t, w.gamma1, w.gamma2)


# ------------------------------------------------------------------ calls ---


def gpu_quant(x_bf16: np.ndarray, bits):
    B, d = x_bf16.shape
    x = dev_bf16(x_bf16)
    codes = torch.full((B, d), 77, dtype=torch.int8, device=DEV)
    scales = torch.full((B,), -1.0, dtype=torch.float32, device=DEV)
    xhat = torch.zeros((B, d), dtype=torch.bfloat16, device=DEV)
    sol.quant_act(x, B, d, dev_i32(bits), codes, scales, xhat)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy(), host_u16(xhat)


def gpu_attention(shape, q_bf16: np.ndarray, kv: DeviceKV, r_permille, ws: Optional[Workspace] = None):
    B, Hq, hd = q_bf16.shape
    Hkv = shape.n_kv_heads
    ws = ws or Workspace(shape, B, kv.max_pages)
    Tmax = kv.max_pages * 64
    out = torch.zeros((B, Hq, hd), dtype=torch.bfloat16, device=DEV)
    kept_idx = torch.full((B, Hkv, Tmax), -1, dtype=torch.int32, device=DEV)
    kept_cnt = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    sol.sparse_decode_attn(shape, dev_bf16(q_bf16), kv.struct(), B, dev_i32(r_permille), out, kept_idx, kept_cnt,
                           ws.buf, ws.bytes)
    torch.cuda.synchronize()
    st = ws.status()
    cnt = kept_cnt.cpu().numpy()
    idx = kept_idx.cpu().numpy()
    kept = [[idx[i, h, : cnt[i, h]] for h in range(Hkv)] for i in range(B)]
    return synth.bf16_to_f32(host_u16(out)).astype(np.float64), kept, st


def gpu_mlp(shape, x_bf16: np.ndarray, w: DeviceWeights, p_permille, ws: Optional[Workspace] = None):
    B, d = x_bf16.shape
    ff = shape.d_ff
    ws = ws or Workspace(shape, B, 1)
    out = torch.zeros((B, d), dtype=torch.bfloat16, device=DEV)
    kept_ch = torch.full((B, ff), -1, dtype=torch.int32, device=DEV)
    kept_cnt = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    t = w.tensors
    sol.pruned_swiglu_mlp(shape, dev_bf16(x_bf16), t["w_gate_up"], t["w_down"], B, dev_i32(p_permille), out,
                          kept_ch, kept_cnt, ws.buf, ws.bytes)
    torch.cuda.synchronize()
    st = ws.status()
    cnt = kept_cnt.cpu().numpy()
    idx = kept_ch.cpu().numpy()
    return synth.bf16_to_f32(host_u16(out)).astype(np.float64), [idx[i, : cnt[i]] for i in range(B)], st


class LayerTaps:
    """Device buffers for every tap of sol_layer_trace_t."""

    def __init__(self, shape, B: int, max_pages: int):
        d, Hq, Hkv, hd, ff = shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff
        f32 = lambda *s: torch.zeros(s, dtype=torch.float32, device=DEV)
        i32 = lambda *s: torch.full(s, -1, dtype=torch.int32, device=DEV)
        i8 = lambda *s: torch.zeros(s, dtype=torch.int8, device=DEV)
        self.t = dict(xn1=f32(B, d), codes1=i8(B, d), scales1=f32(B), q_rot=f32(B, Hq, hd),
                      kept_idx=i32(B, Hkv, max_pages * 64), kept_cnt=i32(B, Hkv), attn_out=f32(B, Hq, hd),
                      h_mid=f32(B, d), xn2=f32(B, d), codes2=i8(B, d), scales2=f32(B), t=f32(B, ff),
                      kept_ch=i32(B, ff), kept_ch_cnt=i32(B), h_out=f32(B, d))
        if shape.quant_placement == sol.QUANT_MLP_OUTPUT:
            self.t.update(z=f32(B, d), z_codes=torch.zeros((B, d), dtype=torch.int16, device=DEV), z_scales=f32(B))
        if shape.mlp_prune == sol.PRUNE_MLP_INPUT:
            self.t.update(xm2=f32(B, d))

    def struct(self):
        return sol.make_trace(**self.t)

    def host(self) -> dict:
        return {k: v.cpu().numpy() for k, v in self.t.items()}


def gpu_layer(shape, w: DeviceWeights, kv: DeviceKV, h_in_bf16: np.ndarray, r, p, b, ws: Optional[Workspace] = None,
              trace=True):
    B, d = h_in_bf16.shape
    ws = ws or Workspace(shape, B, kv.max_pages)
    taps = LayerTaps(shape, B, kv.max_pages) if trace else None
    out = torch.zeros((B, d), dtype=torch.bfloat16, device=DEV)
    sol.decode_layer(shape, w.struct(), kv.struct(), B, dev_bf16(h_in_bf16), out, dev_i32(r), dev_i32(p), dev_i32(b),
                     taps.struct() if taps else None, ws.buf, ws.bytes)
    torch.cuda.synchronize()
    return synth.bf16_to_f32(host_u16(out)).astype(np.float64), (taps.host() if taps else None), ws.status()


# --------------------------------------------------------------- checking ---


def check_token_sets(oshape: O.Shape, sigma, kept_oracle, kept_gpu, seq_lens) -> checker.SetParity:
    tot = checker.SetParity()
    for i in range(len(kept_gpu)):
        forced = O.forced_keep_set(int(seq_lens[i]), oshape.n_sink, oshape.n_window)
        for h in range(oshape.n_kv_heads):
            tot.merge(checker.compare_index_set(sigma[i][h], kept_oracle[i][h], kept_gpu[i][h], forced))
    return tot


def check_channel_sets(t_oracle, kept_oracle, kept_gpu) -> checker.SetParity:
    tot = checker.SetParity()
    for i in range(len(kept_gpu)):
        tot.merge(checker.compare_index_set(np.abs(t_oracle[i]), kept_oracle[i], kept_gpu[i]))
    return tot


def assert_sets(par: checker.SetParity, what: str):
    assert par.ok(), f"{what}: {par}"
    # near-ties are legal but must stay rare
    assert par.near_tie_indices <= max(2, par.sets // 50), f"{what}: too many near-ties {par}"


def assert_outputs(oracle_out, got, what: str):
    m, r = checker.output_errors(oracle_out, got)
    raw_small, raw_all = checker.raw_max_abs(oracle_out, got)
    assert raw_small <= checker.OUT_MAX_ABS, f"{what}: plain max-abs {raw_small:.3e} where |oracle| < 8"
    assert m <= checker.OUT_MAX_ABS and r <= checker.OUT_REL_L2, f"{what}: max-abs {m:.3e} rel-L2 {r:.3e}"
    print(f"{what}: max-abs {raw_all:.3e} plain, {raw_small:.3e} where |oracle| < 8, {m:.3e} in bf16 steps of [4,8); "
          f"rel-L2 {r:.3e}")
    return m, r
