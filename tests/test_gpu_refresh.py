"""GPU parity of the periodic KV-cache refresh (sol_kv_refresh) against the fp64 oracle.

The refreshed cache entries are bf16 numbers that both sides round from their own sums, and from the second layer
on they are computed from the first layer's outputs, so they are compared as numbers: within one bf16 step of the
oracle's entry (2^-7 relative) plus 2e-3 absolute for entries near zero, and nearly all of them bit-equal.  The last
layer's outputs follow the output rule of the decode step (max-abs 2e-2, relative L2 1e-2).
"""
import numpy as np
import pytest
import torch

from oracle import checker
from oracle import sol_oracle as O
from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TINY = dict(synth.WORKLOADS["tiny"], rope_theta=10000.0)


def _case(cfg, n_layers, lens, n, seed, token_select=0, quest_page_size=0):
    shape, oshape = H.make_shapes(cfg, token_select=token_select, quest_page_size=quest_page_size)
    lens = np.asarray(lens, np.int32)
    B = len(lens)
    ws_ = [synth.make_layer_weights(cfg, seed, l) for l in range(n_layers)]
    table, n_pages = synth.make_page_table(lens, True, seed, 0)
    pools = [synth.make_kv_pool(cfg, n_pages, seed, l) for l in range(n_layers)]
    dws = [H.device_weights(w, shape) for w in ws_]
    dkvs = [H.device_kv(k, v, table, lens) for (k, v) in pools]
    h_span = synth.make_hidden(cfg, seed + 1, B * n).reshape(B, n, cfg["d_model"])
    return shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span


def _refresh_gpu(shape, dws, dkvs, B, n, h_span, want_out=True):
    rows = min(B, 128 // n) * n
    ws = H.Workspace(shape, rows, dkvs[0].max_pages)
    out = torch.zeros(h_span.shape, dtype=torch.bfloat16, device=H.DEV) if want_out else None
    sol.kv_refresh(shape, [w.struct() for w in dws], [k.struct() for k in dkvs], B, n, H.dev_bf16(h_span), out, ws.buf,
                   ws.bytes)
    torch.cuda.synchronize()
    return out, ws


def _assert_cache_close(got_u16, want_u16, what):
    g, w = O.bf16_to_f64(got_u16), O.bf16_to_f64(want_u16)
    d = np.abs(g - w)
    assert np.all(d <= np.abs(w) * 2.0 ** -7 + 2e-3), (what, float(d.max()))
    assert np.mean(got_u16 != want_u16) < 0.02, (what, float(np.mean(got_u16 != want_u16)))


def _check_against_oracle(cfg, n_layers, lens, n, seed):
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(cfg, n_layers, lens, n, seed)
    B = len(lens)
    out, ws = _refresh_gpu(shape, dws, dkvs, B, n, h_span)
    assert ws.status()[0] == 0
    okvs = [O.PagedKV(k.copy(), v.copy(), np.where(table < 0, 0, table), lens.copy()) for (k, v) in pools]
    out_o = O.kv_refresh(oshape, [H.oracle_weights(w) for w in ws_], okvs, h_span)
    got = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)
    m, rel = checker.output_errors(out_o.reshape(B * n, -1), got.reshape(B * n, -1))
    assert m <= checker.OUT_MAX_ABS and rel <= checker.OUT_REL_L2, (m, rel)
    for l in range(n_layers):
        _assert_cache_close(H.host_u16(dkvs[l].k_pool), okvs[l].k_pool, f"keys of layer {l}")
        _assert_cache_close(H.host_u16(dkvs[l].v_pool), okvs[l].v_pool, f"values of layer {l}")
        # nothing outside the span was written
        P = 64
        span = np.zeros(pools[l][0].shape[:1] + (P,), bool)
        for i, T in enumerate(lens):
            for t in range(int(T) - n, int(T)):
                span[int(table[i, t // P]), t % P] = True
        same_k = (H.host_u16(dkvs[l].k_pool) == pools[l][0]).all(axis=(1, 3))
        same_v = (H.host_u16(dkvs[l].v_pool) == pools[l][1]).all(axis=(1, 3))
        assert np.all(same_k | span) and np.all(same_v | span)


def test_refresh_sixteen_tokens_two_layers_ragged():
    _check_against_oracle(TINY, 2, [300, 64, 16, 129], 16, seed=3)


@pytest.mark.parametrize("n", [1, 4, 7, 20])
def test_refresh_other_span_lengths(n):
    """Up to 16 tokens the span kernel takes the attention; longer spans go row by row through the decode step's."""
    _check_against_oracle(TINY, 2, [200, 65, n], n, seed=10 + n)


def test_refresh_long_ragged_contexts_split_over_ctas():
    """Contexts of many pages (the span kernel splits them over CTAs), one ending right after a page boundary."""
    _check_against_oracle(TINY, 1, [5000, 1025, 64 * 30 + 1, 17], 16, seed=71)


@pytest.mark.parametrize("hq,hkv", [(4, 1), (2, 2), (8, 1)])
def test_refresh_head_dim_128_and_other_group_sizes(hq, hkv):
    """Two layers, so that the second layer's cache entries depend on the first layer's span attention."""
    cfg = dict(TINY, head_dim=128, n_q_heads=hq, n_kv_heads=hkv)
    _check_against_oracle(cfg, 2, [300, 70, 2049], 16, seed=81)


def test_refresh_group_of_eight_heads_head_dim_64():
    cfg = dict(TINY, n_q_heads=8, n_kv_heads=1)
    _check_against_oracle(cfg, 2, [130, 64, 700], 9, seed=83)


def test_refresh_more_rows_than_one_pass_takes():
    """10 sequences of 16 tokens: the rows go through the layers in passes of 8 and 2 sequences."""
    _check_against_oracle(TINY, 1, [80, 64, 100, 16, 33, 260, 70, 128, 17, 90], 16, seed=21)


def test_refresh_llama1b_layer_shape():
    cfg = dict(synth.WORKLOADS["llama1b_layer"], batch=3)
    _check_against_oracle(cfg, 1, [700, 257, 64], 16, seed=5)


def test_refresh_of_one_token_is_the_dense_decode_step():
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(TINY, 2, [300, 64, 129], 1, 31)
    B = 3
    out, ws = _refresh_gpu(shape, dws, dkvs, B, 1, h_span)
    dkvs2 = [H.device_kv(k, v, table, lens) for (k, v) in pools]
    ws2 = H.Workspace(shape, B, dkvs2[0].max_pages)
    out2 = torch.zeros((B, TINY["d_model"]), dtype=torch.bfloat16, device=H.DEV)
    sol.decode_step(shape, [w.struct() for w in dws], [k.struct() for k in dkvs2], B, H.dev_bf16(h_span[:, 0]), out2,
                    None, H.dev_i32([1000] * B), H.dev_i32([0] * B), H.dev_i32([16] * B), ws2.buf, ws2.bytes)
    torch.cuda.synchronize()
    assert torch.equal(out[:, 0], out2)
    for a, c in zip(dkvs, dkvs2):
        assert torch.equal(a.k_pool, c.k_pool) and torch.equal(a.v_pool, c.v_pool)


def test_refresh_undoes_polluted_decode_steps():
    """Four decode steps under aggressive actions, then the refresh over the same four tokens: the cache comes
    back to what four dense decode steps write (both on the GPU), and the polluted one was different."""
    n, L = 4, 2
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(TINY, L, [300, 68, 129], n, 41)
    B = 3
    dense = [H.device_kv(k, v, table, lens) for (k, v) in pools]
    ws = H.Workspace(shape, B, dkvs[0].max_pages)
    out = torch.zeros((B, TINY["d_model"]), dtype=torch.bfloat16, device=H.DEV)
    for i in range(n):
        step_lens = H.dev_i32(lens - n + 1 + i)
        for kvs, (r, p, b) in ((dkvs, (250, 500, 4)), (dense, (1000, 0, 16))):
            for k in kvs:
                k.seq_lens.copy_(step_lens)
            sol.decode_step(shape, [w.struct() for w in dws], [k.struct() for k in kvs], B, H.dev_bf16(h_span[:, i]),
                            out, None, H.dev_i32([r] * B), H.dev_i32([p] * B), H.dev_i32([b] * B), ws.buf, ws.bytes)
    torch.cuda.synchronize()
    for k in dkvs:
        k.seq_lens.copy_(H.dev_i32(lens))
    assert any(not torch.equal(a.k_pool, c.k_pool) for a, c in zip(dkvs, dense))
    polluted = float(np.abs(O.bf16_to_f64(H.host_u16(dkvs[1].k_pool)) - O.bf16_to_f64(H.host_u16(dense[1].k_pool))).max())
    _refresh_gpu(shape, dws, dkvs, B, n, h_span, want_out=False)
    for l in range(L):
        _assert_cache_close(H.host_u16(dkvs[l].k_pool), H.host_u16(dense[l].k_pool), f"keys of layer {l}")
        _assert_cache_close(H.host_u16(dkvs[l].v_pool), H.host_u16(dense[l].v_pool), f"values of layer {l}")
    assert polluted > 0.05  # the polluted entries were far outside that tolerance


def test_refresh_rebuilds_the_page_extrema_in_quest_mode():
    n = 16
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(TINY, 2, [300, 70, 129], n, 51, token_select=1,
                                                                      quest_page_size=16)
    B = 3
    for k in dkvs:
        k.build_quest_meta(shape, B)
    _refresh_gpu(shape, dws, dkvs, B, n, h_span, want_out=False)
    for k in dkvs:
        got = k.quest_meta.clone()
        k.build_quest_meta(shape, B)  # from the refreshed cache, all pages
        assert torch.equal(got.view(torch.int16), k.quest_meta.view(torch.int16))
    # and the cache is the one the token-selection shape writes: the dense pass does not depend on the mode
    shape0, _ = H.make_shapes(TINY)
    dkvs0 = [H.device_kv(k, v, table, lens) for (k, v) in pools]
    _refresh_gpu(shape0, dws, dkvs0, B, n, h_span, want_out=False)
    for a, c in zip(dkvs, dkvs0):
        assert torch.equal(a.k_pool, c.k_pool) and torch.equal(a.v_pool, c.v_pool)


def test_refresh_refuses_bad_arguments_and_reports_short_sequences():
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(TINY, 1, [100, 64], 4, 61)
    ws = H.Workspace(shape, 128, dkvs[0].max_pages)
    args = ([w.struct() for w in dws], [k.struct() for k in dkvs], 2)
    h = H.dev_bf16(h_span)
    assert sol.kv_refresh(shape, *args, 0, h, None, ws.buf, ws.bytes, check=False) != 0
    assert sol.kv_refresh(shape, *args, 129, h, None, ws.buf, ws.bytes, check=False) != 0
    assert sol.kv_refresh(shape, *args, 4, h, None, ws.buf, 1024, check=False) != 0
    # a sequence shorter than the span: the call runs, stays inside the cache and raises the bad-action bit
    dkvs[0].seq_lens.copy_(H.dev_i32([100, 2]))
    assert sol.kv_refresh(shape, *args, 4, h, None, ws.buf, ws.bytes, check=False) == 0
    torch.cuda.synchronize()
    assert ws.status()[0] & 4


def test_horizon_of_decode_steps_then_refresh_then_decode():
    """The paper's cycle at a small scale: a horizon of decode steps under sparse actions, the refresh over the
    horizon's tokens, then the next decode step.  Each phase is compared with the oracle run on the cache the
    GPU produced so far (a selection may legally differ after a one-ulp difference upstream)."""
    n, L, B = 4, 2, 3
    shape, oshape, ws_, pools, table, lens, dws, dkvs, h_span = _case(TINY, L, [300, 68, 129], n, 91)
    lens_after = lens + 1
    # room for one more token: a page table with a spare slot
    table2, n_pages = synth.make_page_table(lens, True, 91, spare_tokens=1)
    pools = [synth.make_kv_pool(TINY, n_pages, 91, l) for l in range(L)]
    dkvs = [H.device_kv(k, v, table2, lens) for (k, v) in pools]
    ow = [H.oracle_weights(w) for w in ws_]
    ws = H.Workspace(shape, B, dkvs[0].max_pages)
    out = torch.zeros((B, TINY["d_model"]), dtype=torch.bfloat16, device=H.DEV)
    r, p, b = [250, 500, 125], [500, 250, 750], [4, 8, 4]
    for i in range(n):  # the horizon
        step_lens = lens - n + 1 + i
        for k in dkvs:
            k.seq_lens.copy_(H.dev_i32(step_lens))
        host = [k.to_oracle() for k in dkvs]
        sol.decode_step(shape, [w.struct() for w in dws], [k.struct() for k in dkvs], B, H.dev_bf16(h_span[:, i]), out,
                        None, H.dev_i32(r), H.dev_i32(p), H.dev_i32(b), ws.buf, ws.bytes)
        torch.cuda.synchronize()
        okvs = [O.PagedKV(k.k_pool, k.v_pool, k.page_table, step_lens.astype(np.int32)) for k in host]
        out_o, _ = O.decode_step(oshape, ow, okvs, h_span[:, i], r, p, b)
        H.assert_outputs(out_o, synth.bf16_to_f32(H.host_u16(out)).astype(np.float64), f"horizon step {i}")
    # the refresh over the horizon's tokens
    for k in dkvs:
        k.seq_lens.copy_(H.dev_i32(lens))
    host = [k.to_oracle() for k in dkvs]
    _refresh_gpu(shape, dws, dkvs, B, n, h_span, want_out=False)
    okvs = [O.PagedKV(k.k_pool, k.v_pool, k.page_table, lens.copy()) for k in host]
    O.kv_refresh(oshape, ow, okvs, h_span)
    for l in range(L):
        _assert_cache_close(H.host_u16(dkvs[l].k_pool), okvs[l].k_pool, f"keys of layer {l}")
        _assert_cache_close(H.host_u16(dkvs[l].v_pool), okvs[l].v_pool, f"values of layer {l}")
    # the next decode step reads the refreshed cache
    for k in dkvs:
        k.seq_lens.copy_(H.dev_i32(lens_after))
    host = [k.to_oracle() for k in dkvs]
    h_next = synth.make_hidden(TINY, 92, B)
    sol.decode_step(shape, [w.struct() for w in dws], [k.struct() for k in dkvs], B, H.dev_bf16(h_next), out, None,
                    H.dev_i32(r), H.dev_i32(p), H.dev_i32(b), ws.buf, ws.bytes)
    torch.cuda.synchronize()
    assert ws.status()[0] == 0
    okvs = [O.PagedKV(k.k_pool, k.v_pool, k.page_table, lens_after.astype(np.int32)) for k in host]
    out_o, _ = O.decode_step(oshape, ow, okvs, h_next, r, p, b)
    H.assert_outputs(out_o, synth.bf16_to_f32(H.host_u16(out)).astype(np.float64), "step after the refresh")
