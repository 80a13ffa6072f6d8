"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function the header declares, and rejects bad arguments before any
kernel launch."""
import os
import re

import numpy as np
import pytest

from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x1000  # a non-null address that must never be dereferenced on these paths


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sol.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sol_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 14
    lib = sol.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(sol.EXPORTS) == names


def test_status_strings():
    assert sol.status_string(sol.SOL_OK) == "ok"
    assert "workspace" in sol.status_string(sol.SOL_ERR_WORKSPACE_TOO_SMALL)


def _shape(name, **over):
    cfg = dict(synth.WORKLOADS[name], **over)
    return sol.make_shape(cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"])


def test_workspace_sizes():
    for name, cfg in synth.WORKLOADS.items():
        ctx = cfg["context"] or 32768
        n = sol.workspace_bytes(_shape(name), cfg["batch"], (ctx + 64 + 63) // 64)
        assert n > 0 and n % 256 == 0 and n < 8 << 30, (name, n)
    small = sol.workspace_bytes(_shape("tiny"), 4, 8)
    assert sol.workspace_bytes(_shape("tiny"), 4, 16) > small
    assert sol.workspace_bytes(_shape("tiny"), 64, 8) > small
    assert sol.workspace_bytes(_shape("tiny", head_dim=96), 4, 8) == 0
    assert sol.workspace_bytes(_shape("tiny", d_model=300), 4, 8) == 0
    assert sol.workspace_bytes(_shape("tiny", d_ff=1000), 4, 8) == 0
    assert sol.workspace_bytes(_shape("tiny"), 129, 8) == 0
    assert sol.workspace_bytes(_shape("tiny"), 0, 8) == 0


def test_bad_arguments_are_rejected_before_any_launch():
    before = sol.launch_count()
    sh = _shape("tiny")
    kv = sol.make_kv(FAKE, FAKE, FAKE, FAKE, 8, 32)
    assert sol.quant_act(None, 4, 256, FAKE, FAKE, FAKE, check=False) == sol.SOL_ERR_INVALID_ARG
    assert sol.quant_act(FAKE, 4, 12, FAKE, FAKE, FAKE, check=False) == sol.SOL_ERR_UNSUPPORTED
    assert sol.quant_act(FAKE, -1, 256, FAKE, FAKE, FAKE, check=False) == sol.SOL_ERR_INVALID_ARG
    assert sol.sparse_decode_attn(sh, FAKE, kv, 4, FAKE, FAKE, None, None, FAKE, 1024, check=False) \
        == sol.SOL_ERR_WORKSPACE_TOO_SMALL
    assert sol.sparse_decode_attn(sh, None, kv, 4, FAKE, FAKE, None, None, FAKE, 1 << 30, check=False) \
        == sol.SOL_ERR_INVALID_ARG
    bad = _shape("tiny", head_dim=96)
    assert sol.sparse_decode_attn(bad, FAKE, kv, 4, FAKE, FAKE, None, None, FAKE, 1 << 30, check=False) \
        == sol.SOL_ERR_UNSUPPORTED
    assert sol.pruned_swiglu_mlp(sh, FAKE, FAKE, FAKE, 4, FAKE, FAKE, None, None, FAKE, 16, check=False) \
        == sol.SOL_ERR_WORKSPACE_TOO_SMALL
    assert sol.pruned_swiglu_mlp(sh, FAKE, None, FAKE, 4, FAKE, FAKE, None, None, FAKE, 1 << 30, check=False) \
        == sol.SOL_ERR_INVALID_ARG
    w = sol.make_weights(*([FAKE] * 6))
    assert sol.decode_layer(sh, w, kv, 4, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, 64, check=False) \
        == sol.SOL_ERR_WORKSPACE_TOO_SMALL
    w_bad = sol.make_weights(FAKE, FAKE, None, FAKE, FAKE, FAKE)
    assert sol.decode_layer(sh, w_bad, kv, 4, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, 1 << 30, check=False) \
        == sol.SOL_ERR_INVALID_ARG
    assert sol.decode_step(sh, [w], [kv], 200, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE, 1 << 30, check=False) \
        == sol.SOL_ERR_UNSUPPORTED
    # empty batch: nothing to do
    assert sol.decode_layer(sh, w, kv, 0, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, 1 << 30, check=False) == sol.SOL_OK
    assert sol.launch_count() == before


def test_host_entry_validates_actions():
    sh = _shape("tiny")
    kv = sol.make_kv(FAKE, FAKE, FAKE, FAKE, 8, 32)
    w = sol.make_weights(*([FAKE] * 6))
    h = np.zeros((2, 256), np.uint16)
    out = np.zeros((2, 256), np.uint16)
    i32 = lambda *v: np.array(v, np.int32)
    call = lambda r, p, b, l: sol.decode_step_host(sh, [w], [kv], 2, h, out, r, p, b, l, FAKE, 64, check=False)
    assert call(i32(500, 1001), i32(0, 0), i32(8, 8), i32(10, 10)) == sol.SOL_ERR_INVALID_ARG
    assert call(i32(500, 500), i32(0, -1), i32(8, 8), i32(10, 10)) == sol.SOL_ERR_INVALID_ARG
    assert call(i32(500, 500), i32(0, 0), i32(8, 12), i32(10, 10)) == sol.SOL_ERR_UNSUPPORTED
    assert call(i32(500, 500), i32(0, 0), i32(8, 1), i32(10, 10)) == sol.SOL_ERR_INVALID_ARG
    assert call(i32(500, 500), i32(0, 0), i32(8, 8), i32(10, 513)) == sol.SOL_ERR_INVALID_ARG
    assert call(i32(500, 500), i32(0, 0), i32(8, 8), i32(10, 0)) == sol.SOL_ERR_INVALID_ARG
    # valid actions reach the workspace check
    assert call(i32(500, 500), i32(0, 0), i32(8, 16), i32(10, 512)) == sol.SOL_ERR_WORKSPACE_TOO_SMALL


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(sol, "_lib", None)
    monkeypatch.setattr(sol, "LIB_PATH", "/nonexistent/libsol.so")
    with pytest.raises(RuntimeError):
        sol.lib()


def test_packed_weight_sizes_and_rejections():
    """Packed sizes are whole tiles of 128-byte rows; bad arguments are refused before any launch."""
    before = sol.launch_count()
    sh = _shape("llama1b_layer")
    d, ff = 2048, 8192
    assert sol.packed_weight_bytes(sh, sol.W_QKV) == (32 + 16) * 64 * d * 2        # 3072 rows: 24 tiles of 128, no padding
    assert sol.packed_weight_bytes(sh, sol.W_O) == d * d * 2
    assert sol.packed_weight_bytes(sh, sol.W_DOWN) == ff * d * 2
    gu = sol.packed_weight_bytes(sh, sol.W_GATE_UP)
    assert gu >= 2 * ff * d * 2 and gu % (128 * 8) == 0 and gu < 2 * ff * d * 2 * 1.1  # tiles padded to whole rows
    assert sol.packed_weight_bytes(sh, 7) == 0
    assert sol.packed_weight_bytes(_shape("tiny", d_model=300), sol.W_QKV) == 0
    assert sol.pack_weights(sh, sol.W_GATE_UP, FAKE, None, FAKE, gu, check=False) == sol.SOL_ERR_INVALID_ARG
    assert sol.pack_weights(sh, sol.W_DOWN, FAKE, None, FAKE, 16, check=False) == sol.SOL_ERR_WORKSPACE_TOO_SMALL
    assert sol.pack_weights(sh, 9, FAKE, None, FAKE, gu, check=False) == sol.SOL_ERR_INVALID_ARG
    assert sol.launch_count() == before
