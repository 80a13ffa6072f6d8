"""The workspace-free attention entry point against the ordinary one.

Some callers of the library may not allocate device memory on the decode path
(their memory was handed to a pool at start-up, or another runtime owns the
allocator), so sol_sparse_decode_attn_static keeps its scratch in a fixed
array inside the library.  This file checks, through the C ABI, that it gives
the same result as sol_sparse_decode_attn on two calls in a row (the second
with other shapes and rates, so anything the first call left in the shared
array would show), and that a problem larger than the array is refused.
It is named so that pytest collects it last."""
import numpy as np
import pytest
import torch

from oracle import sol_oracle as O
from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def _both(cfg, lens, r, seed, check_free_memory=False):
    shape, oshape = H.make_shapes(cfg)
    lens = np.asarray(lens, np.int32)
    B, Hq, Hkv, hd = len(lens), cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    k_pool, v_pool, table = H.make_case_kv(cfg, lens, seed)
    q = synth.make_queries(cfg, seed, B)
    kv = H.device_kv(k_pool, v_pool, table, lens)
    ref_out, ref_kept, ref_st = H.gpu_attention(shape, q, kv, r)
    Tmax = kv.max_pages * 64
    out = torch.zeros((B, Hq, hd), dtype=torch.bfloat16, device=H.DEV)
    kept_idx = torch.full((B, Hkv, Tmax), -1, dtype=torch.int32, device=H.DEV)
    kept_cnt = torch.full((B, Hkv), -1, dtype=torch.int32, device=H.DEV)
    status = torch.full((8,), -1, dtype=torch.int32, device=H.DEV)
    q_dev, r_dev = H.dev_bf16(q), H.dev_i32(r)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]  # the driver's count of free device memory, not torch's pool
    sol.sparse_decode_attn_static(shape, q_dev, kv.struct(), B, r_dev, out, kept_idx, kept_cnt, status)
    torch.cuda.synchronize()
    if check_free_memory:
        # the entry point's own claim: nothing was allocated (or freed) on the device by the call
        assert torch.cuda.mem_get_info()[0] == free_before
    got = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)
    cnt, idx = kept_cnt.cpu().numpy(), kept_idx.cpu().numpy()
    st = status.cpu().numpy().tolist()
    assert st[0] == 0 and st[1] == 0, st
    assert st[3] == ref_st[3], "both paths re-score the same candidates"
    # same kernels on the same inputs: identical bits, which is inside every tolerance the other tests use
    assert np.array_equal(got, ref_out)
    kept = [[idx[i, h, : cnt[i, h]] for h in range(Hkv)] for i in range(B)]
    for i in range(B):
        for h in range(Hkv):
            assert np.array_equal(kept[i][h], ref_kept[i][h])
    # and against the oracle directly, at the rules of the other attention tests
    okv = O.PagedKV(k_pool, v_pool, np.where(table < 0, 0, table), lens)
    out_o, kept_o, sigma = O.sparse_decode_attn(oshape, O.bf16_to_f64(q), okv, r)
    H.assert_sets(H.check_token_sets(oshape, sigma, kept_o, kept, lens), "token sets of the workspace-free call")
    H.assert_outputs(out_o, got, "output of the workspace-free call")


def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    tiny = synth.WORKLOADS["tiny"]
    _both(tiny, [512, 300, 64, 129], [250, 500, 1000, 125], seed=0)
    # second call: fewer, shorter sequences and other rates reuse the array over the first call's leftovers
    _both(tiny, [65, 200, 1], [500, 125, 1000], seed=1, check_free_memory=True)
    # a third with another head geometry
    _both(dict(synth.WORKLOADS["llama8b_layer"], n_q_heads=8, n_kv_heads=2), [700, 64], [250, 500], seed=2)


def test_static_scratch_refuses_what_does_not_fit():
    cfg = synth.WORKLOADS["llama1b_layer"]  # needs about 30 MB of scratch
    shape, _ = H.make_shapes(cfg)
    before = sol.launch_count()
    fake = 0x1000
    kv = sol.make_kv(fake, fake, fake, fake, 64, 1024)
    s = sol.sparse_decode_attn_static(shape, fake, kv, 16, fake, fake, check=False)
    assert s == sol.SOL_ERR_WORKSPACE_TOO_SMALL
    assert sol.sparse_decode_attn_static(shape, None, kv, 16, fake, fake, check=False) == sol.SOL_ERR_INVALID_ARG
    assert sol.launch_count() == before
