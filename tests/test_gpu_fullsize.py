"""GPU parity at the full sizes of the larger workloads.

The CUDA library runs the whole batch in the launch configuration the
benchmark uses; the fp64 oracle, which cannot afford every sequence at these
sizes, is run on sampled sequences (every step of the path is independent per
sequence, so a sequence's result does not depend on the rest of the batch).

Many-layer steps are checked layer by layer with teacher forcing: every layer
of the step is compared with the oracle on the input that layer really saw on
the GPU (the float32 residual stream tapped between layers, the cache as the
GPU left it), at the rules of test_gpu_parity.py:

  * quantizer codes and scales bit-exact on the GPU's own normalised rows;
  * token and channel index sets equal to the oracle's on the GPU's own
    queries / cache / quantized rows, near-ties (1e-5 relative) counted;
  * each layer's output within max-abs 2e-2 and relative L2 1e-2 of the
    oracle's layer applied to that layer's own inputs.

The end-to-end difference of the whole step (oracle run from the step's input
on its own) is printed, not asserted: a legal one-ulp difference upstream may
legally flip a code or a selection downstream, and the two runs then drift.

The caches of these workloads (up to 27 GB) are drawn on the device by a
seeded generator; the oracle gets the pages of the sampled sequences.
"""
import numpy as np
import pytest
import torch

from oracle import checker
from oracle import sol_oracle as O
from paper_2605_10875_b200 import binding as sol
from paper_2605_10875_b200 import synth
from tests import harness as H
from tests.test_gpu_parity import check_layer, check_stages

pytestmark = pytest.mark.gpu


def test_layer_llama8b_full_size_sampled():
    """One Llama-3.1-8B-shaped layer, batch 64, context 16384 (the fourth workload)."""
    cfg = synth.WORKLOADS["llama8b_layer"]
    r, p, b = synth.draw_actions(cfg, 0)
    lens = synth.make_contexts(cfg, 0)
    # three sequences whose actions differ in every axis
    sample, seen = [], set()
    for i in range(cfg["batch"]):
        key = (int(r[i]), int(p[i]), int(b[i]))
        if all(key[a] != s[a] for s in seen for a in range(3)) or not seen:
            sample.append(i)
            seen.add(key)
        if len(sample) == 3:
            break
    res = check_layer(cfg, lens, r, p, b, sample=sample)
    print("llama8b layer, sampled", sample, res)


# ---------------------------------------------------------------- many layers ---


class SampledStack:
    """L layers on the device at full batch; host copies of the sampled sequences' cache pages, kept in
    step with what the library appended."""

    def __init__(self, cfg, n_layers, start_lens, sample, spare, seed=0):
        self.cfg, self.L, self.sample = cfg, n_layers, np.asarray(sample)
        self.shape, self.oshape = H.make_shapes(cfg)
        self.B = len(start_lens)
        table, n_pages = synth.make_page_table(start_lens, True, seed, spare_tokens=spare)
        self.table = np.where(table < 0, 0, table).astype(np.int32)
        self.max_pages = table.shape[1]
        self.weights = [synth.make_layer_weights(cfg, seed, l) for l in range(n_layers)]
        self.dws = [H.device_weights(w, self.shape) for w in self.weights]
        self.lens_dev = H.dev_i32(start_lens)
        table_dev = H.dev_i32(self.table)
        self.dkvs = []
        for l in range(n_layers):
            k, v = synth.device_kv_pool(cfg, n_pages, H.DEV, seed, l)
            self.dkvs.append(H.DeviceKV(k, v, table_dev, self.lens_dev, self.max_pages, n_pages))
        self.ws = H.Workspace(self.shape, self.B, self.max_pages)
        # compact host pools of the sampled sequences: their pages, renumbered
        need = [(int(start_lens[i]) + spare + 63) // 64 for i in self.sample]
        pages = np.concatenate([self.table[i, :n] for i, n in zip(self.sample, need)])
        self.ctab = np.zeros((len(self.sample), self.max_pages), np.int32)
        at = 0
        for row, n in enumerate(need):
            self.ctab[row, :n] = np.arange(at, at + n)
            at += n
        pidx = torch.from_numpy(pages.astype(np.int64)).to(H.DEV)
        self.host_k = [H.host_u16(kv.k_pool.index_select(0, pidx)) for kv in self.dkvs]
        self.host_v = [H.host_u16(kv.v_pool.index_select(0, pidx)) for kv in self.dkvs]
        self.taps = [H.LayerTaps(self.shape, self.B, self.max_pages) for _ in range(n_layers)]

    def step_and_check(self, lens, h_in, r, p, b, what):
        """One traced step on the GPU, then every layer checked on the sampled sequences."""
        B, idx = self.B, self.sample
        lens = np.asarray(lens, np.int32)
        self.lens_dev.copy_(H.dev_i32(lens))
        out = torch.zeros((B, self.cfg["d_model"]), dtype=torch.bfloat16, device=H.DEV)
        sol.decode_step_traced(self.shape, [w.struct() for w in self.dws], [k.struct() for k in self.dkvs], B,
                               H.dev_bf16(h_in), out, None, H.dev_i32(r), H.dev_i32(p), H.dev_i32(b),
                               [t.struct() for t in self.taps], self.ws.buf, self.ws.bytes)
        torch.cuda.synchronize()
        st = self.ws.status()
        assert st[0] == 0 and st[1] == 0 and st[2] == 0, st
        got = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)[idx]
        rs, ps, bs, ls = np.asarray(r)[idx], np.asarray(p)[idx], np.asarray(b)[idx], lens[idx]
        didx = torch.from_numpy(idx.astype(np.int64)).to(H.DEV)
        h64 = O.bf16_to_f64(h_in[idx])
        summary = dict(near_ties=0, flips=0, e2e_asserted=0, worst_layer_err=(0.0, 0.0))
        # the oracle's own step from the step's input (for the printed end-to-end drift only)
        own_kvs = [O.PagedKV(self.host_k[l].copy(), self.host_v[l].copy(), self.ctab, ls) for l in range(self.L)]
        own_out, _ = O.decode_step(self.oshape, [H.oracle_weights(w) for w in self.weights], own_kvs, h_in[idx], rs, ps, bs)
        for l in range(self.L):
            taps = {key: val.index_select(0, didx).cpu().numpy() for key, val in self.taps[l].t.items()}
            # the cache after this layer: the rows this library appended, brought back for the sampled sequences
            k_after, v_after = self.host_k[l].copy(), self.host_v[l].copy()
            for row, i in enumerate(idx):
                pos = int(lens[i]) - 1
                pg, slot = int(self.table[i, pos // 64]), pos % 64
                cpg = int(self.ctab[row, pos // 64])
                k_after[cpg, :, slot] = H.host_u16(self.dkvs[l].k_pool[pg, :, slot])
                v_after[cpg, :, slot] = H.host_u16(self.dkvs[l].v_pool[pg, :, slot])
            res = check_stages(self.oshape, self.weights[l], h64, self.ctab, ls, rs, ps, bs, taps, self.host_k[l],
                               self.host_v[l], k_after, v_after, out=got if l == self.L - 1 else None, status=st)
            summary["near_ties"] += res["tokens"].near_tie_indices + res["channels"].near_tie_indices
            summary["flips"] += res["code_flips"]
            summary["e2e_asserted"] += int(res["end_to_end_asserted"])
            summary["worst_layer_err"] = tuple(max(a, c) for a, c in zip(summary["worst_layer_err"], res["err"]))
            # later layers and steps read what THIS library produced
            self.host_k[l], self.host_v[l] = k_after, v_after
            h64 = taps["h_out"].astype(np.float64)
        m, rel = checker.output_errors(own_out, got)
        summary["end_to_end_drift"] = dict(max_abs=float(m), rel_l2=float(rel))
        print(what, "sampled", idx.tolist(), "contexts", ls.tolist(), summary, "status", st)
        return summary


def _pick_samples(bits, lens, extra=()):
    """One sequence without a quantizer, one at the coarsest width, the shortest and the longest context, plus `extra`."""
    bits = np.asarray(bits)
    out = [int(np.flatnonzero(bits == 16)[0]), int(np.flatnonzero(bits == bits.min())[0]), int(np.argmin(lens)),
           int(np.argmax(lens))]
    for e in extra:
        if int(e) not in out:
            out.append(int(e))
    return sorted(set(out))


def test_step_llama1b_16_layers_full_size_every_layer():
    """The 16-layer Llama-3.2-1B-shaped step, batch 32, context 8192 (the third workload), at a budget
    of 0.375: the batch mixes the two keep-rates around it.  All 16 layers, four sampled sequences."""
    cfg = synth.WORKLOADS["llama1b_step"]
    r, p, b = synth.budget_mix_actions(cfg, 375, 0)
    # the third workload sweeps r with p = 0; two of the sampled sequences also get a prune rate so that the
    # channel selection is exercised at this batch size
    lens = synth.make_contexts(cfg, 0)
    sample = _pick_samples(b, lens, (np.argmin(r), np.argmax(r)))[:4]
    p = p.copy()
    p[sample[0]], p[sample[-1]] = 500, 250
    stack = SampledStack(cfg, cfg["layers"], lens, sample, spare=0)
    stack.step_and_check(lens, synth.make_hidden(cfg, 0), r, p, b, "llama1b 16-layer step")


def test_ragged_serving_steps_across_an_action_redraw_every_layer():
    """The ragged serving mix: batch 128, lognormal contexts in [256, 32768], all 16 layers, consecutive
    steps that append to the cache: steps 14, 15, 16 of the 64-step cycle, i.e. both sides of the redraw
    of the per-sequence actions (every 16 steps).  Eight sampled sequences, among them the shortest and
    the longest context."""
    cfg = synth.WORKLOADS["ragged_serving"]
    first, steps, redraw_every = 14, 3, 16
    final = synth.make_contexts(cfg, 0)
    start = np.maximum(final - 63, 1).astype(np.int32)  # context at step 0 of the cycle
    b0 = synth.draw_actions(cfg, 0, redraw=0)[2]
    sample = _pick_samples(b0, start, (5, 17, 40, 77, 101))[:8]
    stack = SampledStack(cfg, cfg["layers"], start + first, sample, spare=steps + 1)
    for s in range(first, first + steps):
        lens = (start + s + 1).astype(np.int32)
        r, p, b = synth.draw_actions(cfg, 0, redraw=s // redraw_every)
        stack.step_and_check(lens, synth.make_hidden(cfg, 100 + s), r, p, b, f"ragged serving step {s}")


def _attention_sets_case(cfg, lens, r, extra_sample, label):
    """The stand-alone attention call on a batch of contexts (one layer's cache): kept counts of every sequence,
    index sets and outputs of sampled sequences, among them the shortest and the longest, against the oracle."""
    shape, oshape = H.make_shapes(cfg)
    B, Hq, Hkv, hd = cfg["batch"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    table, n_pages = synth.make_page_table(lens, True, 0)
    tab = np.where(table < 0, 0, table).astype(np.int32)
    k, v = synth.device_kv_pool(cfg, n_pages, H.DEV, 0, 0)
    kv = H.DeviceKV(k, v, H.dev_i32(tab), H.dev_i32(lens), table.shape[1], n_pages)
    q = synth.make_queries(cfg, 0, B)
    Tmax = kv.max_pages * 64
    ws = H.Workspace(shape, B, kv.max_pages)
    out = torch.zeros((B, Hq, hd), dtype=torch.bfloat16, device=H.DEV)
    kept_idx = torch.full((B, Hkv, Tmax), -1, dtype=torch.int32, device=H.DEV)
    kept_cnt = torch.full((B, Hkv), -1, dtype=torch.int32, device=H.DEV)
    sol.sparse_decode_attn(shape, H.dev_bf16(q), kv.struct(), B, H.dev_i32(r), out, kept_idx, kept_cnt, ws.buf, ws.bytes)
    torch.cuda.synchronize()
    st = ws.status()
    assert st[0] == 0 and st[1] == 0, st
    # every sequence: kept counts follow the budget formula
    cnt = kept_cnt.cpu().numpy()
    for i in range(B):
        assert np.all(cnt[i] == O.kept_token_count(int(r[i]), int(lens[i]), 1)), i
    sample = sorted(set([int(np.argmin(lens)), int(np.argmax(lens))] + extra_sample))[:9]
    # compact host cache of the sampled sequences
    need = [(int(lens[i]) + 63) // 64 for i in sample]
    pages = np.concatenate([tab[i, :n] for i, n in zip(sample, need)])
    ctab = np.zeros((len(sample), kv.max_pages), np.int32)
    at = 0
    for row, n in enumerate(need):
        ctab[row, :n] = np.arange(at, at + n)
        at += n
    pidx = torch.from_numpy(pages.astype(np.int64)).to(H.DEV)
    okv = O.PagedKV(H.host_u16(k.index_select(0, pidx)), H.host_u16(v.index_select(0, pidx)), ctab, lens[sample])
    out_o, kept_o, sigma = O.sparse_decode_attn(oshape, O.bf16_to_f64(q[sample]), okv, r[sample])
    idx = kept_idx.cpu().numpy()
    kept = [[idx[i, h, : cnt[i, h]] for h in range(Hkv)] for i in sample]
    par = H.check_token_sets(oshape, sigma, kept_o, kept, lens[sample])
    H.assert_sets(par, label + " token sets")
    got = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)[sample]
    err = H.assert_outputs(out_o, got, label + " attention output")
    print(label, "attention: sampled", sample, "contexts", lens[sample].tolist(), par, "status", st, "err", err)


def test_attention_ragged_batch_128_sets():
    """Ragged batch-128 contexts: the scoring pass numbers the units that exist (flat grid)."""
    cfg = synth.WORKLOADS["ragged_serving"]
    lens = synth.make_contexts(cfg, 0)
    r, _, _ = synth.draw_actions(cfg, 0)
    extra = [int(np.flatnonzero(r == x)[0]) for x in cfg["r_set"]] + [3, 50, 90, 127]
    _attention_sets_case(cfg, lens, r, extra, "ragged")


def test_attention_batch_128_long_contexts_more_units_than_ctas():
    """128 sequences of 15000..16384 tokens: 65536 units of the scoring pass for a grid of 32768 CTAs, so every
    CTA takes two units (the second with the other phase of its copy barriers)."""
    cfg = dict(synth.WORKLOADS["ragged_serving"])
    rng = np.random.default_rng(11)
    lens = rng.integers(15000, 16385, size=cfg["batch"]).astype(np.int32)
    lens[5] = 16384
    r, _, _ = synth.draw_actions(cfg, 0)
    extra = [int(np.flatnonzero(r == x)[0]) for x in cfg["r_set"]][:3] + [127]
    _attention_sets_case(cfg, lens, r, extra, "long contexts")


def test_quest_attention_ragged_batch_128_pages():
    """The paper's Quest selection (page size 16) on the ragged batch of 128 contexts: page counts of every query
    head of every sequence by the budget formula, page sets and outputs of sampled sequences (the shortest and
    the longest among them) against the oracle; rows of up to 2048 pages go through the two-precision select."""
    cfg = synth.WORKLOADS["ragged_serving"]
    S = 16
    shape, oshape = H.make_shapes(cfg, token_select=sol.SELECT_QUEST_PAGES, quest_page_size=S)
    B, Hq, Hkv, hd = cfg["batch"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    lens = synth.make_contexts(cfg, 0)
    r, _, _ = synth.draw_actions(cfg, 0)
    table, n_pages = synth.make_page_table(lens, True, 0)
    tab = np.where(table < 0, 0, table).astype(np.int32)
    k, v = synth.device_kv_pool(cfg, n_pages, H.DEV, 0, 0)
    kv = H.DeviceKV(k, v, H.dev_i32(tab), H.dev_i32(lens), table.shape[1], n_pages)
    kv.build_quest_meta(shape, B)
    q = synth.make_queries(cfg, 0, B)
    ws = H.Workspace(shape, B, kv.max_pages)
    Prow = kv.max_pages * 64 // S
    out = torch.zeros((B, Hq, hd), dtype=torch.bfloat16, device=H.DEV)
    pages = torch.full((B, Hq, Prow), -1, dtype=torch.int32, device=H.DEV)
    cnt = torch.full((B, Hq), -1, dtype=torch.int32, device=H.DEV)
    sol.sparse_decode_attn(shape, H.dev_bf16(q), kv.struct(), B, H.dev_i32(r), out, pages, cnt, ws.buf, ws.bytes)
    torch.cuda.synchronize()
    st = ws.status()
    assert st[0] == 0 and st[1] == 0 and st[5] == 0, st
    cn = cnt.cpu().numpy()
    for i in range(B):
        assert np.all(cn[i] == O.quest_kept_page_count(int(r[i]), int(lens[i]), S, 1)), i
    sample = sorted(set([int(np.argmin(lens)), int(np.argmax(lens))] + [int(np.flatnonzero(r == x)[0]) for x in cfg["r_set"]]
                        + [50, 127]))[:8]
    need = [(int(lens[i]) + 63) // 64 for i in sample]
    pidx = torch.from_numpy(np.concatenate([tab[i, :n] for i, n in zip(sample, need)]).astype(np.int64)).to(H.DEV)
    ctab = np.zeros((len(sample), kv.max_pages), np.int32)
    at = 0
    for row, n in enumerate(need):
        ctab[row, :n] = np.arange(at, at + n)
        at += n
    okv = O.PagedKV(H.host_u16(k.index_select(0, pidx)), H.host_u16(v.index_select(0, pidx)), ctab, lens[sample])
    out_o, kept_o, scores = O.quest_decode_attn(oshape, O.bf16_to_f64(q[sample]), okv, r[sample], S)
    pg = pages.cpu().numpy()
    from oracle import checker
    tot = checker.SetParity()
    for row, i in enumerate(sample):
        forced = np.array([(int(lens[i]) - 1) // S])
        for h in range(Hq):
            tot.merge(checker.compare_index_set(scores[row][h], kept_o[row][h], pg[i, h, : cn[i, h]], forced))
    H.assert_sets(tot, "quest page sets (ragged)")
    got = synth.bf16_to_f32(H.host_u16(out)).astype(np.float64)[sample]
    err = H.assert_outputs(out_o, got, "quest ragged attention output")
    print("quest ragged attention: sampled", sample, "contexts", lens[sample].tolist(), tot, "status", st, "err", err)
