#!/usr/bin/env python
"""Benchmark of the action-conditioned decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole hot path (every layer of the workload) over
one batch of synthetic input.  Prints ONE JSON line (rank 0).  With N > 1
(launched by torch.distributed.run) every rank runs an independent replica of
the step on its own GPU: the path needs no exchange between sequences, so
there is no collective in the data path; the ranks meet only at the barriers
around the timed region and the slowest rank's time is reported.

The default workload is the ragged serving mix (the largest configuration: 16
layers, batch 128, contexts 256..32768, consecutive steps that append, actions
redrawn every 16 steps); the same run also times the other four workloads
compactly (`per_workload`) and a small-batch prune-rate sweep.

`--impl reference` times the CPU oracle on the host cores instead (a
deliberately plain fp64 program; a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_10875_b200 import synth  # noqa: E402

METRIC = "action-conditioned decode steps/s"
UNIT = "steps/s"
HBM_SPEC_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
ROTATE = 4  # distinct copies of weights + cache, cycled so that no step finds its inputs in L2 (--rotate)
SERVE_STEPS = 64   # ragged serving workload: consecutive steps that append before the contexts start over
SERVE_REDRAW = 16  # ... and steps between two draws of the per-sequence actions

DEFAULT_WORKLOAD = "ragged_serving"  # the largest single-GPU configuration
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")


def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the streaming kernels from
    the ncu captures summarised under profiles/: lines of `workload kernel read_bytes write_bytes
    captured_units full_units` (a capture of a scaled-down case carries the units it processed and the
    units of a full launch; traffic is scaled by their ratio).  Absent -> null."""
    table = {}
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                parts = line.split("#")[0].split()
                if len(parts) == 6:
                    wl, k, rd, wr, cu, fu = parts
                    table[(wl, k)] = int((int(rd) + int(wr)) * (float(fu) / float(cu)))
    except OSError:
        pass
    return table


def _plain(o):
    return o.item() if hasattr(o, "item") else str(o)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------
# algorithmic bytes
# ----------------------------------------------------------------------------


def kept_tokens(r_permille, T):
    T = int(T)
    return min(T, max(1, (int(r_permille) * T + 999) // 1000))


def kernel_bytes(cfg, seq_lens, r, union_rows):
    """Bytes each streaming kernel must move per launch (one layer)."""
    d, hq, hkv, hd, ff = cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"]
    k_bytes = sum(hkv * int(T) * hd * 2 for T in seq_lens)
    v_bytes = sum(hkv * kept_tokens(ri, T) * hd * 2 for ri, T in zip(r, seq_lens))
    return {
        "attn_score": k_bytes,
        "attn_gather_v": v_bytes,
        "gemm_qkv": (hq + 2 * hkv) * hd * d * 2,
        "gemm_out_proj": d * hq * hd * 2,
        "gemm_gate_up_swiglu": 2 * ff * d * 2,
        "gemm_down_gathered": union_rows * d * 2,
    }


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._period = period_s
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------
# the GPU arm
# ----------------------------------------------------------------------------


class Replica:
    """Device-resident state of one workload: `rotate` copies of weights and caches.  Weights and caches
    are drawn on the device by a seeded generator (the same shapes and distributions as the host-side
    generators of the parity tests; tens of GB would take minutes to draw on the host)."""

    def __init__(self, cfg, device, seed=0, quest_page_size=0):
        import torch

        from paper_2605_10875_b200 import binding as sol

        self.torch, self.sol, self.cfg, self.device = torch, sol, cfg, device
        self.B, self.L = cfg["batch"], cfg["layers"]
        # the ragged serving workload runs consecutive steps that append: contexts grow by one token per
        # step over a cycle of SERVE_STEPS steps and the actions are redrawn every SERVE_REDRAW steps
        self.serving = cfg.get("context") is None
        self.cycle = SERVE_STEPS if self.serving else 1
        self.seq_lens = synth.make_contexts(cfg, seed)
        if self.serving:
            self.seq_lens = np.maximum(self.seq_lens - (self.cycle - 1), 1).astype(np.int32)
        self.shape = sol.make_shape(cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"],
                                    64, synth.RMS_EPS, cfg.get("rope_theta", 0.0), 0, 1,
                                    token_select=sol.SELECT_QUEST_PAGES if quest_page_size else sol.SELECT_TOKENS,
                                    quest_page_size=quest_page_size)
        table, n_pages = synth.make_page_table(self.seq_lens, cfg.get("shuffle_pages", True), seed,
                                               spare_tokens=self.cycle - 1)
        self.max_pages, self.n_pages = table.shape[1], n_pages
        self.table = self._i32(np.where(table < 0, 0, table))
        self.lens_dev = [self._i32(self.seq_lens + j) for j in range(self.cycle)]
        names = ("w_qkv", "w_o", "w_gate_up", "w_down", "gamma1", "gamma2")
        # enough distinct copies of weights + cache that no step finds its inputs in the 126 MB L2; one
        # copy of a multi-GB workload is already far larger than L2
        hkv, hd, d, ff = cfg["n_kv_heads"], cfg["head_dim"], cfg["d_model"], cfg["d_ff"]
        copy_bytes = self.L * (n_pages * hkv * 64 * hd * 4 + (3 * ff * d + 2 * d * (cfg["n_q_heads"] + hkv) * hd) * 2)
        self.rotate = ROTATE if copy_bytes < (1 << 30) else 1
        self.copy_mb = int(copy_bytes / 1e6)
        self.weights, self.kvs, self._keep = [], [], []
        for l in range(self.L):
            wd = self._pack(synth.device_layer_weights(cfg, device, seed, l))  # load-time step, untimed
            base_w = [wd[n] for n in names]
            base_kv = list(synth.device_kv_pool(cfg, n_pages, device, seed, l))
            per_copy_w, per_copy_kv = [], []
            for c in range(self.rotate):
                ws_ = base_w if c == 0 else [t.clone() for t in base_w]
                kv_ = base_kv if c == 0 else [t.clone() for t in base_kv]
                self._keep += ws_ + kv_
                per_copy_w.append(sol.make_weights(*ws_))
                meta = None
                if quest_page_size:  # page extrema of the paper's Quest selection, built once (a prefill's job) for the
                    # longest contexts of the cycle; every step renews the block of the key it appends
                    meta = torch.zeros(sol.quest_meta_bytes(self.shape, n_pages) // 2, dtype=torch.bfloat16, device=device)
                    self._keep.append(meta)
                    sol.quest_build_meta(self.shape, sol.make_kv(kv_[0], kv_[1], self.table, self.lens_dev[-1],
                                                                 self.max_pages, n_pages, meta), self.B)
                per_copy_kv.append([sol.make_kv(kv_[0], kv_[1], self.table, self.lens_dev[j], self.max_pages, n_pages, meta)
                                    for j in range(self.cycle)])
            self.weights.append(per_copy_w)
            self.kvs.append(per_copy_kv)
        self.ws_bytes = sol.workspace_bytes(self.shape, self.B, self.max_pages)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)
        sol.workspace_init(self.ws, self.ws_bytes)
        self.h_in = self._bf16(synth.make_hidden(cfg, seed))
        self.h_out = torch.zeros((self.B, cfg["d_model"]), dtype=torch.bfloat16, device=device)
        # pinned host buffers for the end-to-end path
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        self.h_in_host = pin(synth.make_hidden(cfg, seed).view(np.int16))
        self.h_out_host = torch.zeros((self.B, cfg["d_model"]), dtype=torch.int16).pin_memory()
        self.lens_host = [pin((self.seq_lens + j).astype(np.int32)) for j in range(self.cycle)]
        torch.cuda.synchronize()

    def _pack(self, plain):
        """The library reads its weights in packed form (sol_pack_weights): done once here, at load time."""
        sol, t = self.sol, self.torch
        out = {"gamma1": plain["gamma1"], "gamma2": plain["gamma2"]}
        for name, kind, a, b in (("w_qkv", sol.W_QKV, "w_qkv", None), ("w_o", sol.W_O, "w_o", None),
                                 ("w_gate_up", sol.W_GATE_UP, "w_gate", "w_up"), ("w_down", sol.W_DOWN, "w_down_t", None)):
            n = sol.packed_weight_bytes(self.shape, kind)
            buf = t.empty(n, dtype=t.uint8, device=self.device)
            sol.pack_weights(self.shape, kind, plain[a], plain[b] if b else None, buf, n)
            out[name] = buf
        t.cuda.synchronize()
        return out

    def _bf16(self, u16):
        t = self.torch
        return t.from_numpy(np.ascontiguousarray(u16).view(np.int16)).to(self.device).view(t.bfloat16)

    def _i32(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(np.asarray(a, np.int32))).to(self.device)

    def set_actions(self, r, p, b, redraws=None):
        """redraws: further (r, p, b) sets the serving workload switches to every SERVE_REDRAW steps."""
        pin = lambda a: self.torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        self.acts, self.acts_host, self.acts_np, self._union = [], [], [], {}
        for (rr, pp, bb) in [(r, p, b)] + list(redraws or []):
            self.acts.append((self._i32(rr), self._i32(pp), self._i32(bb)))
            self.acts_host.append(tuple(pin(np.asarray(x, np.int32)) for x in (rr, pp, bb)))
            self.acts_np.append(tuple(np.asarray(x, np.int32) for x in (rr, pp, bb)))

    def _phase(self, i):
        j = i % self.cycle
        return i % self.rotate, j, (j // SERVE_REDRAW) % len(self.acts)

    def step(self, i):
        c, j, a = self._phase(i)
        r, p, b = self.acts[a]
        self.sol.decode_step(self.shape, [w[c] for w in self.weights], [k[c][j] for k in self.kvs], self.B, self.h_in,
                             self.h_out, None, r, p, b, self.ws, self.ws_bytes)

    def step_host(self, i):
        c, j, a = self._phase(i)
        r, p, b = self.acts_host[a]
        self.sol.decode_step_host(self.shape, [w[c] for w in self.weights], [k[c][j] for k in self.kvs], self.B,
                                  self.h_in_host, self.h_out_host, r, p, b, self.lens_host[j], self.ws, self.ws_bytes)

    def union_rows(self, a=0):
        """Rows of W_down that at least one token keeps under action set `a`, from one traced call of layer 0."""
        if a in self._union:
            return self._union[a]
        t, sol = self.torch, self.sol
        ff = self.cfg["d_ff"]
        kept = t.full((self.B, ff), -1, dtype=t.int32, device=self.device)
        cnt = t.zeros((self.B,), dtype=t.int32, device=self.device)
        out = t.zeros_like(self.h_out)
        r, p, b = self.acts[a]
        sol.decode_layer(self.shape, self.weights[0][0], self.kvs[0][0][0], self.B, self.h_in, out, r, p, b,
                         sol.make_trace(kept_ch=kept, kept_ch_cnt=cnt), self.ws, self.ws_bytes)
        t.cuda.synchronize()
        live = t.zeros((ff + 1,), dtype=t.bool, device=self.device)
        valid = t.arange(ff, device=self.device)[None, :] < cnt[:, None]
        live[t.where(valid, kept, t.full_like(kept, ff)).reshape(-1).long()] = True
        self._union[a] = int(live[:ff].sum().item())
        return self._union[a]

    def bytes_of_steps(self, step_indices):
        """Algorithmic bytes of the given steps (mean per step, and mean per launch of each streaming kernel)."""
        tot, per_kernel = 0.0, {}
        for i in step_indices:
            _, j, a = self._phase(i)
            kb = kernel_bytes(self.cfg, self.seq_lens + j, self.acts_np[a][0], self.union_rows(a))
            tot += self.L * sum(kb.values())
            for k, v in kb.items():
                per_kernel[k] = per_kernel.get(k, 0.0) + v
        n = max(1, len(step_indices))
        return tot / n, {k: v / n for k, v in per_kernel.items()}

    def prepare_refresh(self, n_tokens):
        """Buffers of the periodic KV-cache refresh over the last n_tokens tokens of every sequence."""
        t, sol = self.torch, self.sol
        self.refresh_n = n_tokens
        rows = min(self.B, 128 // n_tokens) * n_tokens
        self.refresh_ws_bytes = sol.workspace_bytes(self.shape, rows, self.max_pages)
        self.refresh_ws = t.empty(self.refresh_ws_bytes, dtype=t.uint8, device=self.device)
        sol.workspace_init(self.refresh_ws, self.refresh_ws_bytes)
        span = synth.make_hidden(self.cfg, 7, self.B * n_tokens)
        self.refresh_h = self._bf16(span).view(self.B, n_tokens, self.cfg["d_model"])

    def refresh(self, i):
        c, j = i % self.rotate, self.cycle - 1
        self.sol.kv_refresh(self.shape, [w[c] for w in self.weights], [k[c][j] for k in self.kvs], self.B,
                            self.refresh_n, self.refresh_h, None, self.refresh_ws, self.refresh_ws_bytes)

    def free(self):
        self.weights = self.kvs = self._keep = self.ws = self.refresh_ws = None
        self.torch.cuda.empty_cache()


def timed_steps(rep, steps, warmup, barrier, fn, count_launches=False):
    """`steps` calls of fn(i) after `warmup`; device time by CUDA events on the launching stream."""
    torch = rep.torch
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    barrier()
    if count_launches:
        rep.sol.launch_count(reset=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    if count_launches:
        rep.launches_timed = rep.sol.launch_count(reset=True)
    barrier()
    return e0.elapsed_time(e1)  # ms


class Ranks:
    """The process-group side of the benchmark: one process per GPU, every rank an independent replica.
    The ranks meet only at barriers and to take the slowest rank's time; `backend` "gloo" with device
    "cpu" runs the same plumbing without a GPU (the multi-process tests)."""

    def __init__(self, backend="nccl", device=None):
        import torch
        import torch.distributed as dist

        self.torch, self.dist = torch, dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device if device is not None else f"cuda:{self.local}"
        if self.world > 1:
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=torch.device(self.device))
            else:
                dist.init_process_group(backend)

    @property
    def is_root(self):
        return self.rank == 0

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()

    def max_over_ranks(self, ms):
        if self.world == 1:
            return ms
        t = self.torch.tensor([ms], dtype=self.torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, steps_per_rank, ms):
        """Steps per second of all ranks together: every rank ran steps_per_rank steps in (at most) ms."""
        return self.world * steps_per_rank / (ms / 1e3)

    def close(self):
        if self.world > 1:
            self.dist.barrier()
            self.dist.destroy_process_group()


def config_dict(workload, cfg, context):
    """The `config` of the JSON line: the same keys and values in both arms."""
    return {"workload": workload, "layers": cfg["layers"], "batch": cfg["batch"], "context": int(context),
            "actions": "per-sequence uniform draw, seed 0",
            "l2": "inputs larger than L2 (rotating copies of weights and KV cache where one copy is under 1 GB)"}


def fractions(byt, t_ms, peak_gbs):
    gbs = byt / t_ms / 1e6
    return {"hbm_gbs": round(gbs, 1), "frac_of_measured": round(gbs / peak_gbs, 4),
            "frac_of_spec_8tbs": round(gbs / HBM_SPEC_GBS, 4)}


def sweep_point(rep, ranks, steps, peak_gbs, label):
    n = min(steps, 300)
    t_ms = ranks.max_over_ranks(timed_steps(rep, n, 5, ranks.barrier, rep.step)) / n
    byt, _ = rep.bytes_of_steps(range(5, 5 + n))
    out = dict(label)
    out.update({"us_per_step": round(1e3 * t_ms, 2), "required_mb": round(byt / 1e6, 1)})
    out.update(fractions(byt, t_ms, peak_gbs))
    return out


def flag_non_monotone(rows, key_fn):
    """Marks sweep rows whose step time is more than 1 % above that of the row with the next larger budget
    (rows given in order of shrinking budget)."""
    for prev, cur in zip(rows, rows[1:]):
        if key_fn(prev) and key_fn(cur) and cur["us_per_step"] > 1.01 * prev["us_per_step"]:
            cur["non_monotone"] = True


def run_ours(args):
    import torch

    from paper_2605_10875_b200 import binding as sol

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    ranks = Ranks("nccl")
    world, rank, local, device = ranks.world, ranks.rank, ranks.local, ranks.device
    barrier, max_over_ranks = ranks.barrier, ranks.max_over_ranks

    sol.lib()
    cfg = dict(synth.WORKLOADS[args.workload])
    if args.batch:
        cfg["batch"] = args.batch
    if args.layers:
        cfg["layers"] = args.layers
    rep = Replica(cfg, device, seed=0)
    r, p, b = synth.draw_actions(cfg, 0)
    redraws = [synth.draw_actions(cfg, 0, redraw=k) for k in range(1, SERVE_STEPS // SERVE_REDRAW)] if rep.serving else None
    rep.set_actions(r, p, b, redraws)
    peak_gbs, peak_kind = measured_peaks()
    traffic = ncu_traffic()

    # --- headline: K steps, inputs resident in HBM ---
    with ClockSampler(local) as clocks:
        ms = max_over_ranks(timed_steps(rep, args.steps, args.warmup, barrier, rep.step, count_launches=True))
    launches = rep.launches_timed
    status = sol.read_device_status(rep.ws)
    ms_per_step = ms / args.steps
    value = ranks.whole_job_rate(args.steps, ms)
    timed = range(args.warmup, args.warmup + args.steps)
    req_bytes, _ = rep.bytes_of_steps(timed)

    # --- the same steps with per-kernel CUDA events (on the launching stream), for the dominant kernel's roofline ---
    prof_steps = min(args.steps, 200)
    sol.timing_enable(True)
    timed_steps(rep, prof_steps, args.warmup, barrier, rep.step)
    rows = sol.timing_collect()
    sol.timing_enable(False)
    _, kb = rep.bytes_of_steps(range(0, args.warmup + prof_steps))
    per_kernel = {}
    n_prof = prof_steps + args.warmup
    for name, n, tot in rows:
        per_kernel[name] = {"launches_per_step": n // n_prof, "us_per_launch": 1e3 * tot / n,
                            "us_per_step": 1e3 * tot / n_prof}
    tot_us = sum(v["us_per_step"] for v in per_kernel.values())
    for v in per_kernel.values():
        v["share"] = round(v["us_per_step"] / tot_us, 4)
        v["us_per_launch"] = round(v["us_per_launch"], 3)
        v["us_per_step"] = round(v["us_per_step"], 3)
    for name, nbytes in kb.items():  # nbytes: one layer's bytes for this kernel; the attention kernels run once per group of sequences
        if name in per_kernel:
            nbytes = nbytes * rep.L / max(1, per_kernel[name]["launches_per_step"])
            per_kernel[name]["bytes_per_launch"] = int(nbytes)
            per_kernel[name]["gbs"] = round(nbytes / per_kernel[name]["us_per_launch"] / 1e3, 1)
            per_kernel[name]["frac_of_measured"] = round(per_kernel[name]["gbs"] / peak_gbs, 4)
    streaming = {k: v for k, v in per_kernel.items() if "bytes_per_launch" in v}
    dom = max(streaming, key=lambda k: streaming[k]["us_per_step"])
    achieved = streaming[dom]["gbs"]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                "frac": round(achieved / peak_gbs, 4), "peak_kind": f"of {peak_kind}",
                "frac_of_spec_8tbs": round(achieved / HBM_SPEC_GBS, 4),
                "bytes_per_launch": streaming[dom]["bytes_per_launch"],
                "traffic": traffic.get((args.workload, dom))}

    # --- end to end: host buffers in, host buffers out, every step ---
    e2e_steps = min(args.steps, 500)
    ms_e2e = max_over_ranks(timed_steps(rep, e2e_steps, 3, barrier, rep.step_host))
    hb = rep.B * cfg["d_model"] * 2
    e2e = {"value": round(ranks.whole_job_rate(e2e_steps, ms_e2e), 2), "unit": UNIT, "steps": e2e_steps,
           "h2d_bytes_per_step": hb + 4 * rep.B * 4, "d2h_bytes_per_step": hb}

    # --- budget sweep: every sequence with the same action ---
    sweep = []
    if not args.no_sweep:
        r_rows, p_rows = [], []
        for (rr, pp, bb) in [(1000, 0, 16), (500, 0, 16), (250, 0, 16), (125, 0, 16), (1000, 250, 16), (1000, 500, 16),
                             (1000, 750, 16), (1000, 0, 8), (1000, 0, 4), (125, 750, 4)]:
            rep.set_actions(*synth.uniform_actions(rep.B, rr, pp, bb))
            row = sweep_point(rep, ranks, args.steps, peak_gbs, {"r": rr / 1000, "p": pp / 1000, "b": bb})
            sweep.append(row)
            if pp == 0 and bb == 16:
                r_rows.append(row)
            if rr == 1000 and bb == 16:
                p_rows.append(row)
        flag_non_monotone(r_rows, lambda x: True)
        flag_non_monotone(p_rows, lambda x: True)
        if sweep[-1]["us_per_step"] > 1.01 * r_rows[-1]["us_per_step"]:  # (r=.125, p=.75, b=4) against (r=.125, p=0)
            sweep[-1]["non_monotone"] = True
        # the same budgets as a batch mix of the two adjacent keep-rates (how a fixed schedule hits a
        # budget that falls between discrete levels), bit-widths drawn per sequence
        mix_rows = []
        for tgt in (1000, 500, 250, 125):
            rep.set_actions(*synth.budget_mix_actions(cfg, tgt, 0))
            mix_rows.append(sweep_point(rep, ranks, args.steps, peak_gbs, {"mix_mean_r": tgt / 1000, "p": 0.0, "b": "drawn"}))
        flag_non_monotone(mix_rows, lambda x: True)
        sweep += mix_rows
        rep.set_actions(r, p, b, redraws)
    context = int(np.max(rep.seq_lens + rep.cycle - 1))
    rotate, copy_mb = rep.rotate, rep.copy_mb
    rep.free()
    del rep

    # --- the other workloads, compactly, and where the prune rate saves bytes (small batches) ---
    per_workload, small_batch = {}, []
    if not args.no_others:
        n = min(args.steps, 100)
        for name in sorted(synth.WORKLOADS):
            if name == args.workload:
                continue
            c2 = synth.WORKLOADS[name]
            rp = Replica(c2, device, seed=0)
            entry = {}
            for tag, acts in (("drawn", synth.draw_actions(c2, 0)), ("dense", synth.uniform_actions(rp.B, 1000, 0, 16)),
                              ("r0.125", synth.uniform_actions(rp.B, 125, 0, 16))):
                rd = [synth.draw_actions(c2, 0, redraw=k) for k in range(1, SERVE_STEPS // SERVE_REDRAW)] \
                    if (rp.serving and tag == "drawn") else None
                rp.set_actions(*acts, rd)
                t_ms = max_over_ranks(timed_steps(rp, n, 5, barrier, rp.step)) / n
                byt, _ = rp.bytes_of_steps(range(5, 5 + n))
                e = {"steps_per_s": round(world * 1e3 / t_ms, 2), "us_per_step": round(1e3 * t_ms, 2),
                     "required_mb": round(byt / 1e6, 1)}
                e.update(fractions(byt, t_ms, peak_gbs))
                entry[tag] = e
            per_workload[name] = entry
            rp.free()
            del rp
        # one Llama-3.2-1B-shaped layer at batch 1 and 4: the union of kept W_down rows is small there
        base = synth.WORKLOADS["llama1b_layer"]
        for bsz in (1, 4):
            c2 = dict(base, batch=bsz)
            rp = Replica(c2, device, seed=0)
            rows_b = []
            for pp in (0, 500, 750):
                rp.set_actions(*synth.uniform_actions(bsz, 1000, pp, 16))
                row = sweep_point(rp, ranks, min(args.steps, 100), peak_gbs, {"batch": bsz, "r": 1.0, "p": pp / 1000, "b": 16})
                row["union_rows"] = rp.union_rows(0)
                # the down projection on its own (event-timed launches): its bytes are the union of kept rows
                sol.timing_enable(True)
                timed_steps(rp, 20, 5, barrier, rp.step)
                trows = {name: 1e3 * tot / n for name, n, tot in sol.timing_collect()}
                sol.timing_enable(False)
                row["down_us_per_launch"] = round(trows.get("gemm_down_gathered", 0.0), 2)
                row["down_mb"] = round(row["union_rows"] * c2["d_model"] * 2 / 1e6, 2)
                rows_b.append(row)
            flag_non_monotone(rows_b, lambda x: True)
            small_batch += rows_b
            rp.free()
            del rp

    # --- the periodic KV-cache refresh: a dense pass over the last tokens of every sequence of the workload ---
    refresh = None
    if args.refresh:
        rf = Replica(cfg, device, seed=0)
        rf.prepare_refresh(args.refresh)
        nr = 3
        t_ms = max_over_ranks(timed_steps(rf, nr, 2, barrier, rf.refresh)) / nr
        sol.timing_enable(True)
        timed_steps(rf, 1, 1, barrier, rf.refresh)
        rows_r = sol.timing_collect()
        sol.timing_enable(False)
        refresh = {"tokens": args.refresh, "ms_per_refresh": round(t_ms, 3),
                   "kernels_us_per_launch": {name: round(1e3 * tot / n, 2) for name, n, tot in rows_r},
                   "kernel_launches_per_refresh": int(sum(n for _, n, _ in rows_r)),
                   "decode_steps_of_the_horizon_ms": round(args.refresh * ms_per_step, 3),
                   "share_of_horizon": round(t_ms / (t_ms + args.refresh * ms_per_step), 4),
                   "tokens_per_s": round(world * 1e3 * rf.B * args.refresh / t_ms, 1),
                   "device_status": sol.read_device_status(rf.refresh_ws)}
        rf.free()
        del rf

    # --- the same workload with the paper's own token sparsity (Quest pages per query head) ---
    quest = None
    if args.quest:
        rq = Replica(cfg, device, seed=0, quest_page_size=args.quest)
        rq.set_actions(r, p, b, redraws)
        nq = min(args.steps, 100)
        t_ms = max_over_ranks(timed_steps(rq, nq, args.warmup, barrier, rq.step)) / nq
        sol.timing_enable(True)
        timed_steps(rq, min(nq, 20), args.warmup, barrier, rq.step)
        rows_q = sol.timing_collect()
        sol.timing_enable(False)
        quest = {"page_size": args.quest, "us_per_step": round(1e3 * t_ms, 2), "steps_per_s": round(world * 1e3 / t_ms, 2),
                 "token_selection_us_per_step": round(1e3 * ms_per_step, 2),
                 "kernels_us_per_launch": {name: round(1e3 * tot / n, 2) for name, n, tot in rows_q
                                           if name.startswith(("quest", "attn_"))},
                 "device_status": sol.read_device_status(rq.ws)}
        rq.free()
        del rq

    line = None
    if rank == 0:
        cpu = None if (world > 1 or args.no_cpu_baseline) else cpu_baseline(args.workload, budget_s=20.0)
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(args.workload, cfg, context),
            "parallelism": "replicas only" if world > 1 else "single GPU",
            "l2_defeat": f"{rotate} rotating cop{'ies' if rotate > 1 else 'y'} of weights and KV cache, {copy_mb} MB each",
            "required_bytes_per_step": int(req_bytes),
            "hbm_tbs": round(req_bytes / ms_per_step / 1e9, 4),
            "hbm_frac_of_measured_peak": round(req_bytes / ms_per_step / 1e6 / peak_gbs, 4),
            "hbm_frac_of_spec_8tbs": round(req_bytes / ms_per_step / 1e6 / HBM_SPEC_GBS, 4),
            "roofline": roofline, "kernels": per_kernel, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks.summary(), "device_status": status,
            "budget_sweep": sweep, "per_workload": per_workload, "small_batch_prune_sweep": small_batch,
            "quest_selection": quest, "kv_refresh": refresh,
        }
        print(json.dumps(line, default=_plain), flush=True)
    ranks.close()
    return line


# ----------------------------------------------------------------------------
# the CPU oracle arm (baseline)
# ----------------------------------------------------------------------------


def _oracle_inputs(cfg, n_seq, seed=0):
    """Inputs of the first n_seq sequences of the workload, one layer, as the oracle takes them."""
    from oracle import sol_oracle as O

    lens = synth.make_contexts(cfg, seed)[:n_seq]
    table, n_pages = synth.make_page_table(lens, cfg.get("shuffle_pages", True), seed)
    k, v = synth.make_kv_pool(cfg, n_pages, seed, 0)
    w = synth.make_layer_weights(cfg, seed, 0)
    ow = O.LayerWeights(w.w_qkv, w.w_o, w.w_gate, w.w_up, w.w_down_t, w.gamma1, w.gamma2)
    shape = O.Shape(cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"], 64,
                    synth.RMS_EPS, cfg.get("rope_theta", 0.0), 0, 1)
    kv = O.PagedKV(k, v, np.where(table < 0, 0, table), lens)
    r, p, b = synth.draw_actions(cfg, seed)
    h = O.bf16_to_f64(synth.make_hidden(cfg, seed)[:n_seq])
    return O, shape, ow, kv, h, r[:n_seq], p[:n_seq], b[:n_seq]


def _host_threads():
    try:
        from threadpoolctl import threadpool_info

        n = [int(i.get("num_threads", 1)) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return 1


def cpu_baseline(workload, budget_s=20.0):
    """Times the oracle, as it stands, on a bounded sample of the workload: one layer over the first
    n sequences, n chosen so the work stays near `budget_s`; scaled to whole steps per second."""
    cfg = synth.WORKLOADS[workload]
    B, L = cfg["batch"], cfg["layers"]
    O, shape, ow, kv, h, r, p, b = _oracle_inputs(cfg, 1)
    t0 = time.perf_counter()
    O.decode_layer(shape, ow, kv, h, r, p, b)
    t1 = time.perf_counter() - t0
    n = int(max(1, min(B, budget_s // max(t1, 1e-3))))
    if n > 1:
        O, shape, ow, kv, h, r, p, b = _oracle_inputs(cfg, n)
        t0 = time.perf_counter()
        O.decode_layer(shape, ow, kv, h, r, p, b)
        t1 = time.perf_counter() - t0
    # a sample that runs in well under the budget is repeated (about 10 s of work in all) and averaged
    reps = int(max(1, min(50, 10.0 // max(t1, 1e-3))))
    if reps > 1:
        t0 = time.perf_counter()
        for _ in range(reps):
            O.decode_layer(shape, ow, kv, h, r, p, b)
        t1 = (time.perf_counter() - t0) / reps
    step_s = t1 * (B / n) * L
    return {"value": round(1.0 / step_s, 6), "unit": UNIT, "cores": _host_threads(), "kind": "oracle",
            "sample": f"one layer over the first {n} of {B} sequences, mean of {reps} run(s) ({t1:.2f} s each), "
                      f"scaled by {B}/{n} sequences x {L} layers"}


def run_reference(args):
    """The oracle as the reference arm: every step is the bounded sample of cpu_baseline."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    cfg = synth.WORKLOADS[args.workload]
    B, L = cfg["batch"], cfg["layers"]
    O, shape, ow, kv, h, r, p, b = _oracle_inputs(cfg, 1)
    t0 = time.perf_counter()
    O.decode_layer(shape, ow, kv, h, r, p, b)
    t1 = time.perf_counter() - t0
    total = args.steps + args.warmup
    n = int(max(1, min(B, (150.0 / total) // max(t1, 1e-3))))
    steps = args.steps
    if n == 1 and t1 * total > 300.0:
        steps = max(1, int(300.0 / t1) - args.warmup)
    O, shape, ow, kv, h, r, p, b = _oracle_inputs(cfg, n)
    for _ in range(args.warmup):
        O.decode_layer(shape, ow, kv, h, r, p, b)
    t0 = time.perf_counter()
    for _ in range(steps):
        O.decode_layer(shape, ow, kv, h, r, p, b)
    dt = (time.perf_counter() - t0) / steps
    step_s = dt * (B / n) * L
    value = round(1.0 / step_s, 6)
    sample = (f"each step: one layer over the first {n} of {B} sequences ({dt:.2f} s), "
              f"scaled by {B}/{n} sequences x {L} layers")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": args.warmup,
            "ms_per_step": round(1e3 * step_s, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": config_dict(args.workload, cfg, int(np.max(synth.make_contexts(cfg, 0)))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": _host_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rotate", type=int, default=ROTATE,
                    help="distinct copies of weights and KV cache cycled through the steps (1 for a small profiler capture)")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (a scaled-down case for a profiler capture)")
    ap.add_argument("--layers", type=int, default=None, help="override the workload's layer count (same purpose)")
    ap.add_argument("--quest", type=int, default=16, choices=[0, 4, 8, 16, 32, 64],
                    help="also time the workload with the paper's Quest page selection at this page size (0: skip)")
    ap.add_argument("--refresh", type=int, default=16,
                    help="tokens per sequence of the timed KV-cache refresh (the paper's horizon T = 16); 0: skip")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the compact runs of the other workloads")
    args = ap.parse_args()
    globals()["ROTATE"] = max(1, args.rotate)
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 128 if args.steps is None else args.steps
        args.warmup = 8 if args.warmup is None else max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
