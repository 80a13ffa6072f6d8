"""GPU parity of the paper's own token sparsity (Quest pages per query head) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import checker
from oracle import sol_oracle as O
from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu

TINY = synth.WORKLOADS["tiny"]
L1B = synth.WORKLOADS["llama1b_layer"]


def _meta_host(kv: H.DeviceKV, shape, S):
    """[num_pages][Hkv][64/S][2][hd] float64 from the device buffer."""
    u16 = H.host_u16(kv.quest_meta)
    return O.bf16_to_f64(u16).reshape(kv.num_pages, shape.n_kv_heads, 64 // S, 2, shape.head_dim)


def _check_meta(meta, okv: O.PagedKV, oshape, S, what):
    """Every block that holds a token: extrema equal to those the oracle takes from the cache rows."""
    B = len(okv.seq_lens)
    for i in range(B):
        T = int(okv.seq_lens[i])
        for kvh in range(oshape.n_kv_heads):
            K = O.cache_rows(okv.k_pool, okv.page_table[i], T, kvh)
            mp, mm = O.quest_page_extrema(K, S)
            for pg in range(len(mp)):
                tok = pg * S
                page = int(okv.page_table[i][tok // 64])
                got = meta[page, kvh, (tok % 64) // S]
                assert np.array_equal(got[0], mp[pg]) and np.array_equal(got[1], mm[pg]), (what, i, kvh, pg)


def _quest_case(cfg, seq_lens, r, S, seed=0, n_sink=0, n_window=1):
    shape, oshape = H.make_shapes(cfg, n_sink, n_window, token_select=sol.SELECT_QUEST_PAGES, quest_page_size=S)
    B = len(seq_lens)
    seq_lens = np.asarray(seq_lens, np.int32)
    Hq = oshape.n_q_heads
    k_pool, v_pool, table = H.make_case_kv(cfg, seq_lens, seed)
    q = synth.make_queries(cfg, seed, B)
    kv = H.device_kv(k_pool, v_pool, table, seq_lens)
    kv.build_quest_meta(shape, B)
    okv = O.PagedKV(k_pool, v_pool, np.where(table < 0, 0, table), seq_lens)
    _check_meta(_meta_host(kv, shape, S), okv, oshape, S, "built extrema")

    ws = H.Workspace(shape, B, kv.max_pages)
    Prow = kv.max_pages * 64 // S
    out = torch.zeros((B, Hq, oshape.head_dim), dtype=torch.bfloat16, device=H.DEV)
    pages = torch.full((B, Hq, Prow), -1, dtype=torch.int32, device=H.DEV)
    cnt = torch.full((B, Hq), -1, dtype=torch.int32, device=H.DEV)
    sol.sparse_decode_attn(shape, H.dev_bf16(q), kv.struct(), B, H.dev_i32(r), out, pages, cnt, ws.buf, ws.bytes)
    torch.cuda.synchronize()
    st = ws.status()
    assert st[0] == 0 and st[1] == 0, st
    out_o, kept_o, scores = O.quest_decode_attn(oshape, O.bf16_to_f64(q), okv, r, S)
    pg, cn = pages.cpu().numpy(), cnt.cpu().numpy()
    tot = checker.SetParity()
    for i in range(B):
        T = int(seq_lens[i])
        forced = np.unique(O.forced_keep_set(T, n_sink, n_window) // S)
        n = O.quest_kept_page_count(int(r[i]), T, S, len(forced))
        for h in range(Hq):
            assert cn[i, h] == n, (i, h, cn[i, h], n)
            got = pg[i, h, :n]
            assert np.all(np.diff(got) > 0), "kept pages must be ascending"
            tot.merge(checker.compare_index_set(scores[i][h], kept_o[i][h], got, forced))
    H.assert_sets(tot, "quest page sets")
    got_out = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)
    err = H.assert_outputs(out_o, got_out, f"quest attention output (S={S})")
    return tot, err


@pytest.mark.parametrize("S", [4, 8, 16, 64])
def test_quest_attention_tiny_workload(S):
    r, _, _ = synth.draw_actions(TINY, 0)
    _quest_case(TINY, synth.make_contexts(TINY, 0), r, S)


@pytest.mark.parametrize("r", [0, 1, 125, 500, 999, 1000])
def test_quest_attention_ragged_lengths_every_rate(r):
    lens = [1, 2, 15, 16, 17, 63, 64, 65, 129, 500, 512]
    _quest_case(TINY, lens, [r] * len(lens), 16, seed=r + 1)


def test_quest_attention_mixed_rates_and_sink_window():
    lens = [300, 77, 512, 5, 200, 64, 33]
    _quest_case(TINY, lens, [250, 500, 125, 1000, 50, 0, 300], 8, seed=3, n_sink=5, n_window=20)


@pytest.mark.parametrize("S", [4, 16])
def test_quest_attention_llama1b_layer_full(S):
    r, _, _ = synth.draw_actions(L1B, 0)
    _quest_case(L1B, synth.make_contexts(L1B, 0), r, S)


def test_quest_attention_head_dim_128():
    cfg = dict(TINY, head_dim=128, n_q_heads=8, n_kv_heads=2)
    _quest_case(cfg, [700, 64, 1, 333], [250, 125, 500, 60], 16, seed=9)


@pytest.mark.parametrize("hq,hkv,S", [(8, 1, 8), (4, 4, 4), (12, 2, 8), (8, 1, 64)])
def test_quest_attention_other_group_sizes(hq, hkv, S):
    cfg = dict(TINY, n_q_heads=hq, n_kv_heads=hkv, d_model=256 if (hq * 64) % 256 == 0 else 768)
    _quest_case(cfg, [333, 64, 190, 700], [250, 500, 125, 60], S, seed=hq)


def test_quest_long_row_many_pages_per_head_pass():
    """A 20000-token row at page size 4: 5000 pages per head, more than one pass of heads through shared memory."""
    _quest_case(TINY, [20000, 4097], [125, 500], 4, seed=21)


def test_quest_page_size_below_group_is_refused():
    cfg = dict(TINY, n_q_heads=8, n_kv_heads=1, d_model=256)
    shape, _ = H.make_shapes(cfg, token_select=sol.SELECT_QUEST_PAGES, quest_page_size=4)
    assert sol.workspace_bytes(shape, 4, 8) == 0
    assert sol.quest_meta_bytes(shape, 16) == 0


def test_quest_layer_updates_extrema_and_matches_oracle():
    """A whole layer step in Quest mode: the appended key enters its block's extrema before the pages are scored,
    and the layer output follows the oracle's layer with the same selection."""
    cfg, S = TINY, 8
    shape, oshape = H.make_shapes(cfg, token_select=sol.SELECT_QUEST_PAGES, quest_page_size=S)
    seq_lens = np.asarray([97, 64, 65, 1, 300, 8], np.int32)
    B = len(seq_lens)
    r = np.asarray([250, 500, 125, 1000, 300, 0], np.int32)
    p = np.zeros(B, np.int32)
    b = np.full(B, 16, np.int32)
    w = synth.make_layer_weights(cfg, 5)
    k_pool, v_pool, table = H.make_case_kv(cfg, seq_lens, 5)
    h_in = synth.make_hidden(cfg, 5, B)
    kv = H.device_kv(k_pool, v_pool, table, seq_lens)
    # extrema of the cache BEFORE the step: every token but the newest (whose key the step writes)
    kv.seq_lens = H.dev_i32(seq_lens - 1)
    kv.build_quest_meta(shape, B)
    kv.seq_lens = H.dev_i32(seq_lens)
    out, _, st = H.gpu_layer(shape, H.device_weights(w, shape), kv, h_in, r, p, b, trace=False)
    assert st[0] == 0 and st[1] == 0 and st[2] == 0, st
    tab = np.where(table < 0, 0, table)
    okv = O.PagedKV(k_pool.copy(), v_pool.copy(), tab, seq_lens)
    ow = H.oracle_weights(w)
    h_o, tr = O.decode_layer(oshape, ow, okv, O.bf16_to_f64(h_in), r, p, b, token_select=O.SELECT_QUEST_PAGES,
                             quest_page_size=S)
    # the cache after the step: the oracle appended to okv; the device extrema must equal those of that cache
    gkv = O.PagedKV(H.host_u16(kv.k_pool), H.host_u16(kv.v_pool), tab, seq_lens)
    _check_meta(_meta_host(kv, shape, S), gkv, oshape, S, "extrema after the append")
    m, rel = checker.output_errors(h_o, out)
    print("quest layer: max-abs", m, "rel-L2", rel)
    assert rel <= checker.OUT_REL_L2, rel
