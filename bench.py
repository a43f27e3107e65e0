#!/usr/bin/env python
"""Benchmark of the MASW hot path on B200: one "step" is one speculative iteration on synthetic
Llama-shaped inputs — gamma draft steps (per layer: raw-KV append, once per iteration the memory-slot
materialisation, draft attention over the compact memory), the verifier's attention over its full
KV cache for every target layer, the accept/reject rule, and the rollback to the starting state.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3_8b_32k] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (a bounded sample).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "draft+verify attention us/step at 32K prefix"
# dram__bytes_read + dram__bytes_write of one launch divided by its KV bytes, from the ncu capture of an 8K-prefix
# case summarised in profiles/attend_kernels_cfg2_full.md (verify: 34.03 MB for 33.575 MB of KV; draft: 4.43 MB for
# 4.19 MB of KV, the rest being q, the pending rows and the split partials)
NCU_TRAFFIC_RATIO = 34.03 / 33.575
NCU_TRAFFIC_RATIO_DRAFT = 4.43 / 4.194
UNIT = "us/step"
TRACE_WORDS = 32   # 64-bit words per CTA in the developer build's stamp records
SMI_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def verify_hint_bytes(wl):
    """Bytes of the next layer's cache a verify launch asks to be brought into L2 (masw_kv_desc.next_k / next_v): per
    CTA tile number `split` and, where a CTA has statically assigned tiles, the first of them (128 entries each, K and
    V).  Averaged over the layers of a step (the last layer has no successor)."""
    heads = wl.batch * wl.t_kv_heads
    splits = max(1, min(148 // heads, 64))
    tiles = (wl.prefix + wl.gamma + 127) // 128
    splits = min(splits, tiles)
    n_static = (max(0, tiles - splits) // 4) // splits
    per_cta = (1 + min(n_static, 1)) * 128 * wl.t_head_dim * 2 * 2
    return splits * heads * per_cta * (wl.t_layers - 1) / wl.t_layers


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# GPU arm
class StepRunner:
    """Owns the resident state (draft memory, target caches, adaptor weights), the per-step input
    staging buffers, and the CUDA graphs of one speculative iteration."""

    def __init__(self, wl, device, seed_offset=0):
        import torch
        from paper_2608_30252_b200 import binding
        self.torch, self.binding, self.wl, self.dev = torch, binding, wl, device
        B, g = wl.batch, wl.gamma
        gen = torch.Generator(device=device)
        gen.manual_seed(260830252 + 1000 * wl.config_id + seed_offset)
        self.gen = gen
        bf = torch.bfloat16

        # ---- resident: draft memory (slots + window filled), adaptor weights, target KV caches
        self.cfg = binding.MaswConfig(wl.d_layers, B, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim, wl.d_model, wl.sink,
                                      wl.window, wl.slot_interval, rollback=wl.rollback, max_slots=wl.slots + 16,
                                      gamma_max=max(8, g))
        self.mem = binding.DraftMemory(self.cfg, device)
        flat = self.mem.arena.view(bf)
        chunk = 1 << 26
        for i in range(0, flat.numel(), chunk):
            flat[i:i + chunk].normal_(generator=gen)
        self.t0 = wl.sink + wl.slots * wl.slot_interval
        self.mem.mem_set_state(t=[self.t0] * B, n_slots=[wl.slots] * B)
        self.t_keep = torch.full((B,), self.t0, dtype=torch.int32, device=device)
        self.m_keep = torch.full((B,), wl.slots, dtype=torch.int32, device=device)
        d, kvw = wl.d_model, wl.d_kv_heads * wl.d_head_dim
        self.Wk = [(torch.randn((d, kvw), generator=gen, device=device) * d ** -0.5).to(bf) for _ in range(wl.d_layers)]
        self.Wv = [(torch.randn((d, kvw), generator=gen, device=device) * d ** -0.5).to(bf) for _ in range(wl.d_layers)]
        cap = wl.prefix + 8
        self.tK, self.tV = [], []
        for _ in range(wl.t_layers):
            k = torch.empty((B, wl.t_kv_heads, cap, wl.t_head_dim), dtype=bf, device=device)
            v = torch.empty_like(k)
            k.normal_(generator=gen); v.normal_(generator=gen)
            self.tK.append(k); self.tV.append(v)
        self.kv_len = torch.full((B,), wl.prefix + g, dtype=torch.int32, device=device)
        self.slot_pos = torch.full((B,), self.t0 + self.slot_step + 1, dtype=torch.int32, device=device)

        # ---- per-step inputs: one packed staging buffer (device) + pinned host mirror
        self.fields = {}
        off = 0

        def field(name, shape, dtype):
            nonlocal off
            n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
            off = (off + 255) // 256 * 256
            self.fields[name] = (off, shape, dtype)
            off += n

        for j in range(g):
            nq = 2 if j == self.slot_step else 1
            field(f"dq{j}", (wl.d_layers, B, nq, wl.d_q_heads, wl.d_head_dim), bf)
            field(f"dk{j}", (wl.d_layers, B, 1, wl.d_kv_heads, wl.d_head_dim), bf)
            field(f"dv{j}", (wl.d_layers, B, 1, wl.d_kv_heads, wl.d_head_dim), bf)
        field("hg", (wl.d_layers, B, d), bf)
        field("vq", (wl.t_layers, B, g, wl.t_q_heads, wl.t_head_dim), bf)
        field("tl", (B, g + 1, wl.vocab), bf)
        field("toks", (B, g), torch.int32)
        self.in_bytes = (off + 255) // 256 * 256
        self.dev_in = torch.empty(self.in_bytes, dtype=torch.uint8, device=device)
        self.host_in = torch.empty(self.in_bytes, dtype=torch.uint8).pin_memory()
        self._fill_host_inputs()
        self.dev_in.copy_(self.host_in)
        self.e2e_graph = None   # captured by the first end-to-end step

        # ---- outputs
        self.d_o1 = torch.empty((wl.d_layers, B, 1, wl.d_q_heads, wl.d_head_dim), dtype=torch.float32, device=device)
        self.d_lse1 = torch.empty((wl.d_layers, B, 1, wl.d_q_heads), dtype=torch.float32, device=device)
        self.d_o2 = torch.empty((wl.d_layers, B, 2, wl.d_q_heads, wl.d_head_dim), dtype=torch.float32, device=device)
        self.d_lse2 = torch.empty((wl.d_layers, B, 2, wl.d_q_heads), dtype=torch.float32, device=device)
        self.v_o = torch.empty((wl.t_layers, B, g, wl.t_q_heads, wl.t_head_dim), dtype=torch.float32, device=device)
        self.v_lse = torch.empty((wl.t_layers, B, g, wl.t_q_heads), dtype=torch.float32, device=device)
        # the decision of a step: accepted lengths [B], then emitted tokens [B][g + 1], in one buffer (one copy back)
        self.out_dev = torch.empty((B * (g + 2),), dtype=torch.int32, device=device)
        self.n_acc = self.out_dev[:B]
        self.out_tok = self.out_dev[B:].view(B, g + 1)
        self.host_out = torch.empty((B * (g + 2),), dtype=torch.int32).pin_memory()
        self.out_bytes = self.host_out.numel() * 4
        self.v_ws = binding.verify_workspace(self.tK[0], self.kv_len, wl.t_q_heads, g)
        self.a_ws = binding.accept_workspace(B, g, wl.vocab, device)
        self.graphs = None
        self.launches_per_step = 0

    @property
    def slot_step(self):
        """The draft step of each iteration on which the memory-slot materialisation fires."""
        return min(2, self.wl.gamma - 1)

    def view(self, name):
        off, shape, dtype = self.fields[name]
        n = int(np.prod(shape)) * self.torch.empty((), dtype=dtype).element_size()
        return self.dev_in[off:off + n].view(dtype).view(shape)

    def _fill_host_inputs(self):
        torch = self.torch
        g = torch.Generator()
        g.manual_seed(12345 + self.wl.config_id)
        for name, (off, shape, dtype) in self.fields.items():
            n = int(np.prod(shape))
            if name == "toks":
                t = torch.randint(0, self.wl.vocab, shape, generator=g, dtype=torch.int32)
            elif name == "tl":
                t = (torch.randn(shape, generator=g) * 4.0).to(dtype)
            else:
                t = torch.randn(shape, generator=g).to(dtype)
            self.host_in[off:off + n * t.element_size()].copy_(t.view(torch.uint8).reshape(-1))

    # ---- the three phases of one speculative iteration, as C-ABI calls on the current stream
    def draft_phase(self, steps=None):
        wl, mem = self.wl, self.mem
        for j in (range(wl.gamma) if steps is None else steps):
            fire = (j == self.slot_step)
            q, k, v = self.view(f"dq{j}"), self.view(f"dk{j}"), self.view(f"dv{j}")
            for l in range(wl.d_layers):
                if fire:   # boundary step: append + slot materialisation + attention (raw row and slot row) in one launch
                    mem.draft_boundary_attend(l, k[l], v[l], self.view("hg")[l], self.Wk[l], self.Wv[l], self.slot_pos, q[l],
                                              out=self.d_o2[l], lse=self.d_lse2[l])
                else:
                    mem.draft_append_attend(l, k[l], v[l], q[l], out=self.d_o1[l], lse=self.d_lse1[l])
            # noted on the host only: the launches that follow and the rollback take it as launch parameters, so no
            # counter kernel sits between draft steps and the next step's first layer may run ahead like the others
            mem.mem_advance(1, add_slot=fire, deferred=True)

    def verify_phase(self):
        wl = self.wl
        vq = self.view("vq")
        for l in range(wl.t_layers):
            # the caches are resident and static here: no kernel in the stream writes them (stable_cache)
            self.binding.verify_attend(self.tK[l], self.tV[l], self.kv_len, vq[l], workspace=self.v_ws, out=self.v_o[l],
                                       lse=self.v_lse[l], stable_cache=True,
                                       next_kv=(self.tK[l + 1], self.tV[l + 1]) if l + 1 < wl.t_layers else None)

    def tail_phase(self):
        self.binding.accept_reject(self.view("tl"), None, self.view("toks"), None, 0.0, workspace=self.a_ws,
                                   n_accepted=self.n_acc, out_tokens=self.out_tok)
        self.mem.mem_rollback(self.t_keep, self.m_keep, slots_keep_max=self.wl.slots)

    def capture(self):
        torch = self.torch
        # eager warm-up of every entry point (sets kernel attributes, builds descriptors) before capture
        self.draft_phase(); self.verify_phase(); self.tail_phase()
        torch.cuda.synchronize()
        graphs = []
        l0 = self.binding.launch_count()
        for phase in (self.draft_phase, self.verify_phase, self.tail_phase):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                phase()
            graphs.append(g)
        self.launches_per_step = self.binding.launch_count() - l0
        self.graphs = graphs
        self.step_graph = None
        torch.cuda.synchronize()
        _, _, status = self.mem.mem_get_state()
        assert status == 0, f"device status word {status}"

    def capture_step(self):
        """The whole iteration as one graph: what the timed steps replay (the per-phase graphs give the breakdown)."""
        torch = self.torch
        self.step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.step_graph):
            self.draft_phase(); self.verify_phase(); self.tail_phase()
        torch.cuda.synchronize()

    def step_resident(self, events=None):
        """One iteration with inputs already in HBM: one graph launch, or, with CUDA events between the phases,
        one graph launch per phase."""
        if events is None:
            if self.step_graph is None:
                self.capture_step()
            self.step_graph.replay()
            return
        for i, g in enumerate(self.graphs):
            if events is not None:
                events[i].record()
            g.replay()
        if events is not None:
            events[3].record()

    def capture_e2e(self):
        """The end-to-end iteration as ONE CUDA graph: the pinned host -> device copies of the step's inputs (on a
        forked copy stream, one copy per phase in the order the phases read them; a phase depends on its own copy
        only, so all but the first draft step's inputs cross the bus while earlier stages run), the three phases,
        and the device -> host copy of the decision."""
        torch = self.torch
        copy_stream = torch.cuda.Stream(device=self.dev)
        # copies in the order they are needed: the first draft step's inputs, the other draft steps' (and h_g), the
        # verifier's queries, the logits and proposals
        first = self.fields["dq1"][0] if (self.wl.gamma > 1 and self.slot_step > 0) else self.fields["vq"][0]
        cuts = [0, first, self.fields["vq"][0], self.fields["tl"][0], self.in_bytes]
        events = [torch.cuda.Event() for _ in range(4)]
        rest = range(1, self.wl.gamma) if first != cuts[2] else range(0)
        stages = [lambda: self.draft_phase(range(0, 1) if first != cuts[2] else None),
                  lambda: self.draft_phase(rest), self.verify_phase, self.tail_phase]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            main = torch.cuda.current_stream()
            copy_stream.wait_stream(main)
            with torch.cuda.stream(copy_stream):
                for a, b, ev in zip(cuts[:-1], cuts[1:], events):
                    if b > a:
                        self.dev_in[a:b].copy_(self.host_in[a:b], non_blocking=True)
                    ev.record(copy_stream)
            for stage, ev in zip(stages, events):
                main.wait_event(ev)
                stage()
            self.host_out.copy_(self.out_dev, non_blocking=True)
            main.wait_stream(copy_stream)
        self.e2e_graph = g
        torch.cuda.synchronize()

    def step_e2e(self):
        """One iteration through host buffers (one graph launch: copies in, the three phases, the decision out),
        then a stream synchronisation: the host holds the step's result when this returns."""
        if self.e2e_graph is None:
            self.capture_e2e()
        self.e2e_graph.replay()
        self.torch.cuda.current_stream().synchronize()


def draft_comparators(wl, device, reps=20):
    """The same draft kernel on the two memories the paper compares against (Section 5.1): the full KV cache
    (window = prefix, no slots) and a sliding window alone (no slots).  Three layers alternate so that no
    launch finds its entries in L2; returns microseconds per layer and launch for each."""
    import torch
    from paper_2608_30252_b200 import binding
    out = {}
    n_layers = 3
    for name, window in (("full_kv", wl.prefix), ("window_only", wl.window)):
        cfg = binding.MaswConfig(n_layers, wl.batch, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim, wl.d_model, 0, window, 1 << 30,
                                 rollback=wl.rollback, max_slots=0, gamma_max=8)
        mem = binding.DraftMemory(cfg, device)
        mem.arena.view(torch.bfloat16).normal_()
        mem.mem_set_state(t=[wl.prefix] * wl.batch, n_slots=[0] * wl.batch)
        q = torch.randn((wl.batch, 1, wl.d_q_heads, wl.d_head_dim), device=device).to(torch.bfloat16)
        k = torch.randn((wl.batch, 1, wl.d_kv_heads, wl.d_head_dim), device=device).to(torch.bfloat16)
        o = torch.empty((wl.batch, 1, wl.d_q_heads, wl.d_head_dim), dtype=torch.float32, device=device)
        lse = torch.empty((wl.batch, 1, wl.d_q_heads), dtype=torch.float32, device=device)
        g = torch.cuda.CUDAGraph()
        s = torch.cuda.Stream(device=device)
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            for l in range(n_layers):
                mem.draft_append_attend(l, k, k, q, out=o, lse=lse)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=s):
                for l in range(n_layers):
                    mem.draft_append_attend(l, k, k, q, out=o, lse=lse)
        torch.cuda.current_stream().wait_stream(s)
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (reps * n_layers)
        mem.close()
        del mem
        torch.cuda.empty_cache()
    return out


def draft_launch_kinds(runner, reps=30):
    """Microseconds per launch of each kind of draft launch, each timed as a CUDA graph of one pass over all draft
    layers in the product library: `plain` = draft_append_attend following another layer's launch (the common
    case: it runs ahead of its predecessor), `plain_after_counter_update` = the same with mem_advance(0) before
    every launch (each launch then reads everything behind its wait, as the first layer of a draft step does),
    `boundary` = draft_boundary_attend following another layer's launch."""
    torch = runner.torch
    wl, mem = runner.wl, runner.mem
    q1, q2 = runner.view("dq0"), runner.view(f"dq{runner.slot_step}")
    k, v = runner.view("dk0"), runner.view("dv0")

    def plain():
        for l in range(wl.d_layers):
            mem.draft_append_attend(l, k[l], v[l], q1[l], out=runner.d_o1[l], lse=runner.d_lse1[l])

    def plain_dirty():
        for l in range(wl.d_layers):
            mem.mem_advance(0)
            mem.draft_append_attend(l, k[l], v[l], q1[l], out=runner.d_o1[l], lse=runner.d_lse1[l])

    def advance_only():
        for l in range(wl.d_layers):
            mem.mem_advance(0)

    def boundary():
        for l in range(wl.d_layers):
            mem.draft_boundary_attend(l, k[l], v[l], runner.view("hg")[l], runner.Wk[l], runner.Wv[l], runner.slot_pos, q2[l],
                                      out=runner.d_o2[l], lse=runner.d_lse2[l])

    out = {}
    side = torch.cuda.Stream(device=runner.dev)
    for name, fn in (("plain", plain), ("plain_after_counter_update", plain_dirty), ("counter_update_alone", advance_only),
                     ("boundary", boundary)):
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            fn()
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (reps * wl.d_layers)
    out["plain_after_counter_update"] -= out.pop("counter_update_alone")
    runner.mem.mem_rollback(runner.t_keep, runner.m_keep, slots_keep_max=wl.slots)
    return out


def reduce_max_over_ranks(values, device=None):
    """Max over ranks of each timing in `values` (replicas run independently; the slowest rank defines
    the job).  Works with any initialised process group (nccl on GPUs, gloo on CPUs); without one the
    values are returned unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_value_us(step_ms_max_over_ranks, world):
    """Whole-job microseconds per step: `world` replicas each finish one step in the slowest rank's time."""
    return step_ms_max_over_ranks * 1e3 / world


class ClockSampler:
    """nvidia-smi polling the SM clock and the throttle reasons every 50 ms.  It is started ahead of the timed
    region (the tool needs a few hundred ms to come up) and `wait_first` lets the caller keep the GPU under the
    same load until the first line has arrived; `begin` / `end` bracket the timed region, and the report uses
    the samples taken inside it (or, if the region was shorter than one period, the last ones before it, taken
    under the warm-up load, and says so)."""

    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        import threading
        self.lines, self.t0, self.t1 = [], None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={SMI_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line))

    def wait_first(self, keep_busy, limit_s=5.0):
        """Runs `keep_busy()` (one more warm-up step) until the first sample is in, for at most `limit_s`."""
        tic = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - tic < limit_s:
            keep_busy()

    def begin(self):
        self.t0 = time.perf_counter()

    def end(self):
        self.t1 = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        t0 = self.t0 if self.t0 is not None else 0.0
        t1 = self.t1 if self.t1 is not None else time.perf_counter()
        inside = [l for ts, l in self.lines if t0 <= ts <= t1 + 0.05]
        where = "timed region"
        if not inside:
            inside = [l for ts, l in self.lines if ts < t0][-3:]
            where = "warm-up load just before the timed region (region shorter than the sampling period)"
        sm, smmax, reasons = [], [], set()
        for line in inside:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smmax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smmax) if smmax else None,
                "samples": len(sm), "sampled_during": where, "reasons": sorted(reasons)}


def oracle_sample(wl, layers_d=1, layers_t=1, seed=7):
    """The CPU oracle, as it stands, on a bounded sample of the workload: `layers_d` draft layers of one
    draft step, `layers_t` target layers of verification, and the accept/reject rule.  Returns the
    measured seconds of each part and the time of a full step scaled linearly by layer count."""
    import oracle
    from paper_2608_30252_b200 import inputs
    rng = np.random.default_rng(seed)
    B, g = wl.batch, wl.gamma
    f64 = oracle.bf16_bits_to_f64
    mem = oracle.DraftMemory(layers_d, B, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim, wl.sink, wl.window, wl.slot_interval)
    t0 = wl.sink + wl.slots * wl.slot_interval
    for l in range(layers_d):
        mem.load_slots(l, f64(inputs.normal_bf16(rng, (B, wl.slots, wl.d_kv_heads, wl.d_head_dim))),
                       f64(inputs.normal_bf16(rng, (B, wl.slots, wl.d_kv_heads, wl.d_head_dim))))
        kw = f64(inputs.normal_bf16(rng, (wl.sink + wl.window, wl.d_kv_heads, wl.d_head_dim)))
        for b in range(B):
            # only the sink and the last W raw tokens are ever read: the tokens between are placeholders
            raw = [None] * t0
            for i in range(wl.sink):
                raw[i] = (kw[i], kw[i])
            for i in range(wl.window):
                raw[t0 - wl.window + i] = (kw[wl.sink + i], kw[wl.sink + i])
            mem.raw[l][b] = raw
    mem.t = [t0] * B
    mem.M = [wl.slots] * B
    d = wl.d_model
    Wk = f64(inputs.normal_bf16(rng, (d, wl.d_kv_heads * wl.d_head_dim), d ** -0.5))
    hg = f64(inputs.normal_bf16(rng, (B, d)))
    q = f64(inputs.normal_bf16(rng, (B, 1, wl.d_q_heads, wl.d_head_dim)))
    kr = f64(inputs.normal_bf16(rng, (B, 1, wl.d_kv_heads, wl.d_head_dim)))
    tic = time.perf_counter()
    for l in range(layers_d):
        mem.append_raw(l, kr, kr)
        mem.attend(l, q)
    t_draft = time.perf_counter() - tic
    tic = time.perf_counter()
    for l in range(layers_d):
        mem.materialize(l, hg, Wk, Wk, [t0 + 1] * B)
    t_slot = time.perf_counter() - tic
    K = f64(inputs.normal_bf16(rng, (B, wl.t_kv_heads, wl.prefix + g, wl.t_head_dim)))
    V = f64(inputs.normal_bf16(rng, (B, wl.t_kv_heads, wl.prefix + g, wl.t_head_dim)))
    vq = f64(inputs.normal_bf16(rng, (B, g, wl.t_q_heads, wl.t_head_dim)))
    tic = time.perf_counter()
    for _ in range(layers_t):
        oracle.verify_attend(vq, K, V, [wl.prefix + g] * B)
    t_verify = time.perf_counter() - tic
    tl, _ = inputs.logits_pair(rng, B, g, wl.vocab)
    toks = f64(tl)[:, :g].argmax(-1)
    tic = time.perf_counter()
    oracle.accept_reject(f64(tl), None, toks, np.zeros((B, g + 1), np.float32), 0.0)
    t_accept = time.perf_counter() - tic
    full = (t_draft / layers_d * wl.d_layers * g + t_slot / layers_d * wl.d_layers
            + t_verify / layers_t * wl.t_layers + t_accept)
    return {"draft_s": t_draft, "slot_s": t_slot, "verify_s": t_verify, "accept_s": t_accept,
            "measured_s": t_draft + t_slot + t_verify + t_accept, "full_step_s": full}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def cpu_baseline(wl, budget_s=20.0):
    probe = oracle_sample(wl, 1, 1)
    per = max(probe["measured_s"], 1e-3)
    n = int(max(1, min(wl.d_layers, wl.t_layers, budget_s / per)))
    res = oracle_sample(wl, n, n) if n > 1 else probe
    # repeat the sample until about 10 s of CPU work are measured (at most 6 passes) and average
    runs = [res]
    while sum(r["measured_s"] for r in runs) < 10.0 and len(runs) < 6:
        runs.append(oracle_sample(wl, n, n))
    value = statistics.mean(r["full_step_s"] for r in runs)
    measured = sum(r["measured_s"] for r in runs)
    return {"value": value * 1e6, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": (f"{n} of {wl.d_layers} draft layers of one draft step + {n} of {wl.t_layers} target layers of "
                       f"verification + accept/reject, {len(runs)} passes, {measured:.1f} s measured in all, scaled "
                       f"linearly by layer count to a full step ({wl.gamma} draft steps)")}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(wl, 1, 1)
    vals = []
    steps = max(1, min(args.steps, 5))
    for _ in range(steps):
        vals.append(oracle_sample(wl, 1, 1)["full_step_s"] * 1e6)
    v = statistics.mean(vals)
    line = {
        "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 1),
        "ms_per_step": v / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "impl": "reference",
        "config": {"workload": wl.name, "prefix": wl.prefix, "gamma": wl.gamma, "batch": wl.batch},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": "each step times 1 draft layer of one draft step, 1 target layer and accept/reject, "
                                   "scaled linearly by layer count to a full step"},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_gpu(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2608_30252_b200 import binding, build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    build.build()
    binding.load()

    runner = StepRunner(wl, dev, seed_offset=rank)
    runner.capture()
    K, W = args.steps, max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- breakdown by phase: blocks of K steps replayed as one graph per phase, with CUDA events between them.
    # Measured first, while only the per-phase graphs exist: once further graphs of the same kernels have been
    # captured in the process, the per-phase replays run about 1 % slower (measured; the whole-step graph does not).
    def phase_warm():
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        runner.step_resident(e)
    for _ in range(W):
        phase_warm()
    phase_blocks, phase_total = [], []
    for _ in range(3):
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
        barrier()
        for i in range(K):
            runner.step_resident(evs[i])
        barrier()
        phase_blocks.append([sum(e[i].elapsed_time(e[i + 1]) for e in evs) / K for i in range(3)])
        phase_total.append(sum(phase_blocks[-1]))
    phase_ms = phase_blocks[sorted(range(3), key=lambda i: phase_total[i])[1]]

    # ---- resident timing: the whole iteration as one graph; W warm-up steps, then blocks of exactly K timed steps
    runner.capture_step()
    clocks = ClockSampler(local) if rank == 0 else None
    for _ in range(W):
        runner.step_resident()
    if clocks is not None:   # more warm-up steps until the clock sampler is up
        clocks.wait_first(lambda: (runner.step_resident(), torch.cuda.synchronize()))
    barrier()
    # The block of exactly K steps is repeated until about half a second has been timed (so that the clock
    # sampler has samples inside the region); the reported step time is the median block, with the spread beside it.
    probe0, probe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    probe0.record(); runner.step_resident(); probe1.record(); barrier()
    n_blocks = int(min(40, max(1, round(args.min_timed_s * 1e3 / max(probe0.elapsed_time(probe1) * K, 1e-3)))))
    if world > 1:   # every rank must run the same number of blocks
        nb = torch.tensor([n_blocks], dtype=torch.int64, device=dev)
        dist.all_reduce(nb, op=dist.ReduceOp.MAX)
        n_blocks = int(nb.item())
    block_ms = []
    if clocks is not None:
        clocks.begin()
    for _ in range(n_blocks):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for i in range(K):
            runner.step_resident()
        stop.record()
        barrier()
        block_ms.append(start.elapsed_time(stop))
    if clocks is not None:
        clocks.end()
    clock_info = clocks.stop() if rank == 0 else None
    order = sorted(range(n_blocks), key=lambda i: block_ms[i])
    mid = order[(n_blocks - 1) // 2]
    total_ms = block_ms[mid]
    block_stats = {"blocks": n_blocks, "steps_per_block": K, "us_per_step_median": block_ms[mid] * 1e3 / K,
                   "us_per_step_min": min(block_ms) * 1e3 / K, "us_per_step_max": max(block_ms) * 1e3 / K,
                   "timed_s": sum(block_ms) / 1e3}

    # ---- end-to-end timing through host buffers
    for _ in range(W):
        runner.step_e2e()
    barrier()
    tic = time.perf_counter()
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    es.record()
    for _ in range(K):
        runner.step_e2e()
    ee.record()
    barrier()
    e2e_ms = es.elapsed_time(ee)
    e2e_wall_ms = (time.perf_counter() - tic) * 1e3
    # the decision the host received is the one on the device, and an accepted length is in range
    assert torch.equal(runner.host_out, runner.out_dev.cpu()), "end-to-end step: host copy of the decision differs"
    assert 0 <= int(runner.host_out[: wl.batch].min()) and int(runner.host_out[: wl.batch].max()) <= wl.gamma
    _, _, status = runner.mem.mem_get_state()

    total_ms, e2e_ms = reduce_max_over_ranks([total_ms, e2e_ms], device=dev)

    if rank == 0:
        step_ms = total_ms / K
        g = wl.gamma
        draft_bytes_step = wl.draft_kv_bytes_per_layer() * wl.d_layers          # one draft step, all layers
        verify_bytes_layer = wl.verify_kv_bytes_per_layer()
        verify_bytes = verify_bytes_layer * wl.t_layers
        draft_us = phase_ms[0] * 1e3 / g
        verify_us = phase_ms[1] * 1e3
        peak, peak_kind = measured_peak_gbs()
        v_gbs = verify_bytes / (verify_us * 1e-6) / 1e9
        d_gbs = draft_bytes_step / (draft_us * 1e-6) / 1e9
        draft_bytes_layer = wl.draft_kv_bytes_per_layer()
        draft_launch_us = draft_us / wl.d_layers               # mean over plain, boundary and first-of-step launches
        step_bytes = draft_bytes_step * g + verify_bytes
        step_gbs = step_bytes / (step_ms * 1e-3) / 1e9
        base = cpu_baseline(wl) if world == 1 and not args.no_cpu_baseline else None
        comp = None
        kinds = draft_launch_kinds(runner) if world == 1 else None
        if world == 1:
            launches_per_step, in_bytes, out_bytes = runner.launches_per_step, runner.in_bytes, runner.out_bytes
            del runner
            torch.cuda.empty_cache()
            comp = draft_comparators(wl, dev)
        else:
            launches_per_step, in_bytes, out_bytes = runner.launches_per_step, runner.in_bytes, runner.out_bytes
        line = {
            "metric": METRIC, "value": job_value_us(step_ms, world), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": step_ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 in / fp32 accumulate", "data": "synthetic",
            "config": {"workload": wl.name, "prefix": wl.prefix, "gamma": g, "batch": wl.batch,
                       "draft": f"{wl.d_layers}L {wl.d_q_heads}q/{wl.d_kv_heads}kv d{wl.d_head_dim}, "
                                f"{wl.slots} slots + {wl.window} window + {wl.sink} sink (r={wl.slot_interval})",
                       "target": f"{wl.t_layers}L {wl.t_q_heads}q/{wl.t_kv_heads}kv d{wl.t_head_dim}, full KV",
                       "step": f"{g} draft steps (slot materialisation on one of them) + verify of {g} rows + "
                               f"greedy accept/reject (V={wl.vocab}) + rollback; replicas only at n_gpus > 1",
                       "l2": "inputs larger than L2 (step reads %.2f GB of KV)" % ((draft_bytes_step * g + verify_bytes) / 1e9),
                       "e2e_step": "one CUDA graph per step: pinned host -> device copies on a forked copy stream in the order "
                                   "they are needed (first draft step's inputs, the other draft steps', the verifier's "
                                   "queries, logits and proposals; a stage depends on its own copy only), the three "
                                   "phases, one copy of the decision device -> host; the host synchronises after every step"},
            "phases": {"draft_us_per_draft_step": draft_us, "draft_us_per_layer": draft_us / wl.d_layers,
                       "draft_kv_gbs": d_gbs, "draft_frac_of_8tbs": d_gbs / 8000.0, "draft_frac_of_measured": d_gbs / peak,
                       "draft_kv_bytes_per_step": draft_bytes_step,
                       "full_kv_draft_bytes_per_step": wl.draft_kv_bytes_per_layer(wl.prefix) * wl.d_layers,
                       "verify_us_per_step": verify_us, "verify_us_per_layer": verify_us / wl.t_layers,
                       "verify_kv_gbs": v_gbs, "verify_frac_of_8tbs": v_gbs / 8000.0,
                       "accept_rollback_us": phase_ms[2] * 1e3},
            "roofline": {"kernel": "attend_tc_kernel (verify_attend, one target layer per launch)", "bound": "hbm",
                         "achieved": v_gbs, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                         "frac": v_gbs / peak, "frac_of_8tbs": v_gbs / 8000.0,
                         "traffic": args.traffic_bytes if args.traffic_bytes
                         else verify_bytes_layer * NCU_TRAFFIC_RATIO + verify_hint_bytes(wl),
                         "traffic_source": "ncu dram bytes of an 8K-prefix launch (profiles/attend_kernels_cfg2_full.md): the "
                                           "launch's own bytes scaled by KV bytes (x 1.014, traffic grows in proportion to the "
                                           "entries) + the next layer's first tiles it asks into L2 (%.1f MB per launch, which "
                                           "the next launch then does not read from DRAM)" % (verify_hint_bytes(wl) / 1e6),
                         "algorithmic_bytes_per_launch": verify_bytes_layer,
                         "launches_timed": wl.t_layers * K * 3,   # the three breakdown blocks
                         "avg_launch_us": verify_us / wl.t_layers},
            # the other half of the step: the draft's decode launch (16.8 MB of KV per launch at batch 1, latency-bound)
            "roofline_draft": {"kernel": "attend_draft_kernel (draft_append_attend / draft_boundary_attend, one draft layer per launch)",
                               "bound": "hbm", "achieved": d_gbs, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                               "frac": d_gbs / peak, "frac_of_8tbs": d_gbs / 8000.0,
                               "traffic": draft_bytes_layer * NCU_TRAFFIC_RATIO_DRAFT,
                               "traffic_source": "ncu dram bytes of an 8K-prefix launch (profiles/attend_kernels_cfg2_full.md) "
                                                 "scaled by KV bytes",
                               "algorithmic_bytes_per_launch": draft_bytes_layer,
                               "launches_timed": wl.d_layers * g * K * 3, "avg_launch_us": draft_launch_us},
            # the whole iteration against the same peak: all KV bytes of the step over the step time
            "step_frac": {"kv_bytes_per_step": step_bytes, "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                          "frac": step_gbs / peak, "frac_of_8tbs": step_gbs / 8000.0},
            "timing": block_stats,
            "e2e": {"value": job_value_us(e2e_ms / K, world), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
                    "d2h_bytes_per_step": out_bytes, "wall_us_per_step": e2e_wall_ms * 1e3 / K},
            "gpu_launches": launches_per_step * K * n_blocks,     # kernels launched inside the timed blocks
            "gpu_launches_per_step": launches_per_step,
            "clocks": clock_info,
            "device_status": status,
        }
        if kinds is not None:
            line["phases"]["draft_us_per_launch_by_kind"] = kinds
        if comp is not None:
            # the paper's comparison points for the draft side (Section 5.1, Table 3), same kernel, one launch per layer
            line["phases"]["draft_comparators_us_per_layer"] = {
                "masw": draft_us / wl.d_layers, "full_kv": comp["full_kv"], "window_only": comp["window_only"]}
            # Eq. 1's cost side from the measured attention times alone (backbone layers are out of scope): draft
            # step cost over verification cost, and the iteration time L_draft * t_d + t_t relative to a full-KV draft
            t_t = verify_us
            c_masw = draft_us / t_t
            c_full = comp["full_kv"] * wl.d_layers / t_t
            line["eq1_attention_only"] = {
                "l_draft": g, "t_d_over_t_t": {"masw": c_masw, "full_kv": c_full},
                "iteration_cost_in_t_t": {"masw": g * c_masw + 1.0, "full_kv": g * c_full + 1.0},
                "iteration_time_vs_full_kv_draft": (g * c_masw + 1.0) / (g * c_full + 1.0)}
            line["phases"]["draft_comparators_kv_bytes_per_layer"] = {
                "masw": wl.draft_kv_bytes_per_layer(), "full_kv": wl.draft_kv_bytes_per_layer(wl.prefix),
                "window_only": wl.draft_kv_bytes_per_layer(wl.window)}
        if base is not None:
            line["cpu_baseline"] = base
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """The sweep configuration: prefix x batch x gamma x slot interval on 8B-target / 1B-draft shapes.  Each
    point is timed with two draft and two target layers (per-layer time does not depend on the layer
    count) and reported per layer and scaled to the nominal 16 / 32 layers.  One JSON line per point."""
    import dataclasses
    import torch
    from paper_2608_30252_b200 import build, binding, inputs
    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build()
    binding.load()
    peak, _ = measured_peak_gbs()
    grid = inputs.sweep_workloads(prefixes=(4096, 8192, 16384, 32768), batches=(1, 4, 16), gammas=(2, 5, 8),
                                  intervals=(20, 8, 4))
    rows = []
    for full in grid:
        wl = dataclasses.replace(full, d_layers=2, t_layers=2)
        runner = StepRunner(wl, dev)
        runner.capture()
        for _ in range(3):
            runner.step_resident()
        torch.cuda.synchronize()
        K = args.steps if args.steps < 100 else 10
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
        for i in range(K):
            runner.step_resident(evs[i])
        torch.cuda.synchronize()
        ph = [sum(e[i].elapsed_time(e[i + 1]) for e in evs) / K for i in range(3)]
        d_layer_us = ph[0] * 1e3 / wl.gamma / wl.d_layers
        v_layer_us = ph[1] * 1e3 / wl.t_layers
        row = {"prefix": wl.prefix, "batch": wl.batch, "gamma": wl.gamma, "slot_interval": wl.slot_interval,
               "memory_entries": wl.draft_entries, "memory_ratio": wl.draft_entries / wl.prefix,
               "draft_us_per_layer": d_layer_us, "draft_us_per_step_16_layers": d_layer_us * full.d_layers,
               "draft_kv_gbs": wl.draft_kv_bytes_per_layer() / (d_layer_us * 1e-6) / 1e9,
               "verify_us_per_layer": v_layer_us, "verify_us_per_step_32_layers": v_layer_us * full.t_layers,
               "verify_kv_gbs": wl.verify_kv_bytes_per_layer() / (v_layer_us * 1e-6) / 1e9,
               "verify_frac_of_measured": wl.verify_kv_bytes_per_layer() / (v_layer_us * 1e-6) / 1e9 / peak,
               "draft_kv_bytes_per_step": wl.draft_kv_bytes_per_layer() * full.d_layers,
               "full_kv_draft_bytes_per_step": wl.draft_kv_bytes_per_layer(wl.prefix) * full.d_layers}
        rows.append(row)
        print(json.dumps(row), flush=True)
        del runner
        torch.cuda.empty_cache()
    return rows


def measured_peak_tflops():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1590.0, 1400.0, "fallback"


def prefill_flops(P, S, W, r, Hq, D):
    """Algorithmic flops of one layer's masked prefill pass: 4 D per (query row, head, visible entry)."""
    M = (P - S) // r if P > S else 0
    t = range(P)
    raw = sum(min(S, x + 1) + ((x - S) // r if x >= S else 0) + (x - max(S, x + 1 - W) + 1 if x >= S else 0) for x in t)
    slot = 0
    for m in range(1, M + 1):
        tau = S + m * r - 1
        slot += S + m + (tau - max(S, tau + 1 - W) + 1)
    return 4.0 * D * Hq * (raw + slot), M


def run_prefill(args, wl):
    """The draft's masked prefill pass at the workload's draft shape: one JSON line with ms per layer and
    the achieved tensor throughput against the measured bf16 peak (a dense contraction: tensor-bound)."""
    import torch
    from paper_2608_30252_b200 import build, binding
    if not torch.cuda.is_available():
        raise RuntimeError("the prefill benchmark needs a CUDA device")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build()
    binding.load()
    B, Hq, Hkv, D = wl.batch, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim
    S, W, r, P = wl.sink, wl.window, wl.slot_interval, wl.prefix
    flops, M = prefill_flops(P, S, W, r, Hq, D)
    flops *= B
    n_layers = 2                                    # two layers' inputs alternate; each layer's q + K/V exceed L2
    cfg = binding.MaswConfig(n_layers, B, Hq, Hkv, D, Hq * D, S, W, r, rollback=16, max_slots=max(M, 1),
                             gamma_max=min(8, 64 // (Hq // Hkv) - 1))
    mem = binding.DraftMemory(cfg, device=dev)
    gen = torch.Generator(device=dev).manual_seed(260830252 + 7)
    q = [torch.randn((B, P + M, Hq, D), generator=gen, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    k = [torch.randn((B, Hkv, P + M, D), generator=gen, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    v = [torch.randn((B, Hkv, P + M, D), generator=gen, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    o = torch.empty((B, P + M, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, P + M, Hq), dtype=torch.float32, device=dev)

    def layer(l):
        mem.draft_prefill_attend(l, k[l], v[l], q[l], P, lse=lse, out_bf16=o, import_memory=True, want_fp32=False)

    sampler = ClockSampler(0)
    for i in range(max(args.warmup, 3)):
        layer(i % n_layers)
    sampler.wait_first(lambda: (layer(0), torch.cuda.synchronize()))
    torch.cuda.synchronize()
    K = min(args.steps, 20)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    l0 = binding.launch_count()
    sampler.begin()
    evs[0].record()
    for i in range(K):
        layer(i % n_layers)
        evs[i + 1].record()
    torch.cuda.synchronize()
    sampler.end()
    launches = binding.launch_count() - l0
    clocks = sampler.stop()
    ms = sum(evs[i].elapsed_time(evs[i + 1]) for i in range(K)) / K
    burst, sustained, kind = measured_peak_tflops()
    tflops = flops / (ms * 1e-3) / 1e12
    _, _, status = mem.mem_get_state()
    row = {"metric": "draft masked prefill ms per layer", "value": ms, "unit": "ms/layer", "n_gpus": 1, "steps": K,
           "warmup": max(args.warmup, 3), "higher_is_better": False, "dtype": "bf16 in / fp32 accumulate",
           "data": "synthetic", "vs_baseline": None,
           "config": {"workload": wl.name + " draft shape", "prefix": P, "slots": M, "window": W, "sink": S,
                      "slot_interval": r, "batch": B, "heads": f"{Hq}q/{Hkv}kv d{D}",
                      "step": "one layer: masked attention of P + M rows, then import of sinks, slots and ring into the arena",
                      "l2": "two layers' inputs alternate (each larger than L2)"},
           "roofline": {"kernel": "prefill_tc_kernel", "bound": "tensor", "achieved": tflops, "peak": sustained,
                        "peak_kind": f"of {kind} (sustained bf16; burst {burst})", "unit": "TFLOP/s",
                        "frac": tflops / sustained, "algorithmic_flops_per_launch": flops, "traffic": None},
           "gpu_launches": launches, "status": status, "clocks": clocks}
    print(json.dumps(row), flush=True)


def run_fp8(args):
    """The verifier's attention over the paged cache in bf16 and in FP8 (e4m3 pages, one scale per page and KV head):
    microseconds per target layer at 32K prefix on the 8B target shape for batch 1, 4 and 16, each timed as a CUDA
    graph over several layers' pools (more bytes than L2).  One JSON line per batch size."""
    import torch
    from paper_2608_30252_b200 import build, binding
    if not torch.cuda.is_available():
        raise RuntimeError("the FP8 comparison needs a CUDA device")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build()
    binding.load()
    peak, _ = measured_peak_gbs()
    Hq, Hkv, D, P, T = 32, 8, 128, 32768, 5
    for B in (1, 4, 16):
        L = 4 if B < 16 else 2
        max_pages = (P + T + 127) // 128
        n_pages = B * max_pages
        gen = torch.Generator(device=dev).manual_seed(260830252 + B)
        table = torch.randperm(n_pages, device=dev, generator=gen).to(torch.int32).view(B, max_pages).contiguous()
        kv_len = torch.full((B,), P + T, dtype=torch.int32, device=dev)
        q = torch.randn((B, T, Hq, D), device=dev, generator=gen).to(torch.bfloat16)
        o = torch.empty((B, T, Hq, D), dtype=torch.float32, device=dev)
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=dev)
        res = {}
        for kind in ("bf16", "fp8"):
            if kind == "bf16":
                Ks = [torch.randn((n_pages, Hkv, 128, D), device=dev, generator=gen).to(torch.bfloat16) for _ in range(2 * L)]
                call = lambda l, ws: binding.verify_attend_paged(Ks[2 * l], Ks[2 * l + 1], table, kv_len, q, workspace=ws, out=o, lse=lse)
            else:   # random bytes below the NaN pattern stand in for quantised values: timing does not depend on them
                Ks = [torch.randint(0, 0x7E, (n_pages, Hkv, 128, D), device=dev, dtype=torch.uint8, generator=gen) for _ in range(2 * L)]
                sc = torch.full((n_pages, Hkv), 0.01, device=dev)
                call = lambda l, ws: binding.verify_attend_fp8(Ks[2 * l], Ks[2 * l + 1], sc, sc, table, kv_len, q, workspace=ws, out=o, lse=lse)
            ws = call(0, None)[2]
            for l in range(L):
                call(l, ws)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for l in range(L):
                        call(l, ws)
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(3):
                g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            res[kind] = e0.elapsed_time(e1) * 1e3 / (10 * L)
            del Ks
            torch.cuda.empty_cache()
        entries_bytes = 2 * (P + T) * Hkv * D * B
        print(json.dumps({"metric": "verify attention us per target layer, paged cache, 32K prefix", "batch": B, "rows": T,
                          "bf16_us": res["bf16"], "fp8_us": res["fp8"], "fp8_speedup": res["bf16"] / res["fp8"],
                          "bf16_kv_gbs": entries_bytes * 2 / (res["bf16"] * 1e-6) / 1e9,
                          "fp8_kv_gbs": entries_bytes / (res["fp8"] * 1e-6) / 1e9, "hbm_peak_gbs": peak,
                          "cache_bytes_per_layer": {"bf16": entries_bytes * 2, "fp8": entries_bytes}}), flush=True)


def run_loop(args):
    """The packaged speculative-decoding loop (paper_2608_30252_b200.loop) on its toy one-layer models: greedy
    decoding of 256 tokens after a 2000-token prompt, gamma = 5, draft memory S = 4, W = 256, r = 8.  Prints one JSON
    line: emitted tokens per iteration, the measured draft-step and verification times, the target's one-token
    time, Eq. 1 evaluated on those measurements, and whether the output equals target-only greedy decoding."""
    import torch
    from paper_2608_30252_b200 import build, binding, loop
    if not torch.cuda.is_available():
        raise RuntimeError("the loop benchmark needs a CUDA device")
    torch.cuda.set_device(0)
    build.build()
    binding.load()
    gamma, n, P = 5, 256, 2000
    g0 = torch.Generator(device="cuda").manual_seed(5)
    prompt = [int(x) for x in torch.randint(0, 64, (P,), generator=g0, device="cuda").tolist()]
    mk_t = lambda: loop.ToyTarget(torch.Generator(device="cuda").manual_seed(1), cap=P + n + 64)
    mk_d = lambda seed: loop.ToyDraft(torch.Generator(device="cuda").manual_seed(seed), S=4, W=256, r=8, max_pos=P + n + 64)
    l0 = binding.launch_count()
    ar_timer = loop.EventTimer()
    ref = loop.greedy_target_only(mk_t(), prompt, n, timer=ar_timer)
    t_ar = ar_timer.mean_us()
    rows = {}
    for name, draft, spoil in (("independent_random_draft", mk_d(7), None),
                               ("draft_right_four_times_in_five", mk_d(7), True)):
        res = loop.speculative(mk_t(), draft, prompt, n, gamma) if spoil is None else \
            _run_spoiled(loop, mk_t(), draft, prompt, n, gamma, ref)
        rows[name] = {"tok_per_iter": res.tok_per_iter, "t_d_us": res.t_d_us, "t_t_us": res.t_t_us,
                      "eq1_speedup": res.eq1_speedup, "iterations": len(res.accepted),
                      "equals_target_only_greedy": res.tokens == ref, "status": res.status}
    print(json.dumps({"metric": "speculative-decoding loop on toy models", "unit": "tokens per iteration / us", "n_gpus": 1,
                      "config": {"workload": "toy 1-layer target (8q/2kv d128) + toy 1-layer MASW draft (8q/2kv d64, S=4 W=256 r=8)",
                                 "prompt": P, "new_tokens": n, "gamma": gamma},
                      "target_one_token_us": t_ar, "drafts": rows, "gpu_launches": binding.launch_count() - l0,
                      "note": "t_d and t_t include the toy models' dense layers (torch matmuls) and host-side launch gaps: "
                              "the loop is driven eagerly from Python, so these times are launch-bound and say nothing "
                              "about the kernels' bandwidth"}), flush=True)


def _run_spoiled(loop, target, draft, prompt, n, gamma, ref):
    """The draft's proposals replaced by the true continuation except every fifth one (a draft that is right four
    times in five), so that Tok./Iter and Eq. 1 are exercised at a realistic acceptance rate."""
    state = {"count": 0}

    def spoil(it, j, tok):
        # position of this proposal in the emitted sequence: reconstructed from the target's cache length
        pos = target.n - len(prompt) + 1 + j
        truth = ref[pos] if pos < len(ref) else 0
        state["count"] += 1
        return (truth + 1) % 64 if state["count"] % 5 == 0 else truth

    return loop.speculative(target, draft, prompt, n, gamma, spoil=spoil)


def run_timeline(args, wl):
    """Per-CTA phase timelines of one draft launch, one boundary launch and one verify launch of `wl`, from
    the %globaltimer stamps of the library's developer hook (eager launches, microseconds from the first
    CTA's start).  Prints one JSON line per launch kind."""
    import numpy as np
    import torch
    from paper_2608_30252_b200 import build, binding
    if not torch.cuda.is_available():
        raise RuntimeError("the timeline needs a CUDA device")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build_trace()
    binding.select_trace_build()      # the stamps exist only in the developer build of the library
    r = StepRunner(wl, dev)
    for _ in range(2):
        r.draft_phase(); r.verify_phase(); r.tail_phase()
    torch.cuda.synchronize()
    n_cta_max = 160
    buf = torch.zeros(n_cta_max * TRACE_WORDS, dtype=torch.int64, device=dev)

    def capture(fn, name, slots, reps=5):
        acc = []
        for _ in range(reps):
            buf.zero_()
            binding.debug_set_trace(buf)
            torch.cuda.synchronize()
            fn()
            torch.cuda.synchronize()
            binding.debug_set_trace(None)
            t = buf.cpu().numpy().reshape(-1, TRACE_WORDS)
            t = t[t[:, 4] > 0]
            t0 = t[:, 0].min()
            acc.append((t[:, [s_ for _, s_ in slots]] - t0) / 1000.0)
        rel = np.stack(acc[1:])          # the first repetition warms the caches of the launch itself
        row = {"launch": name, "ctas": int(rel.shape[1]), "unit": "us from the first CTA's start"}
        for k, (label, _) in enumerate(slots):
            col = rel[:, :, k]
            row[label] = {"median": round(float(np.median(col)), 2), "min": round(float(col.min(axis=1).mean()), 2),
                          "max": round(float(col.max(axis=1).mean()), 2)}
        print(json.dumps(row), flush=True)

    def capture_chain(n_launch=6, reps=4, boundary=False):
        """Consecutive draft layers replayed from one CUDA graph, one record area per launch: when each launch's
        CTAs start, pass their wait, finish their tiles, publish and end, in microseconds from the first launch's
        first CTA (what overlaps between dependent launches shows here, not in a single eager launch)."""
        stride = n_cta_max * TRACE_WORDS
        cbuf = torch.zeros(n_launch * stride, dtype=torch.int64, device=dev)
        q, k, v = r.view(f"dq{r.slot_step}" if boundary else "dq0"), r.view("dk0"), r.view("dv0")
        layers = [l % wl.d_layers for l in range(n_launch)]

        def launch(l):
            if boundary:
                r.mem.draft_boundary_attend(l, k[l], v[l], r.view("hg")[l], r.Wk[l], r.Wv[l], r.slot_pos, q[l],
                                            out=r.d_o2[l], lse=r.d_lse2[l])
            else:
                r.mem.draft_append_attend(l, k[l], v[l], q[l], out=r.d_o1[l], lse=r.d_lse1[l])

        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            r.mem.mem_advance(0)                  # the first launch of the chain follows a counter update, as in a draft step
            for l in layers:
                launch(l)
            torch.cuda.synchronize()
            binding.debug_set_trace(cbuf, stride)
            with torch.cuda.graph(g, stream=side):
                r.mem.mem_advance(0)
                for l in layers:
                    launch(l)
            binding.debug_set_trace(None)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(reps):
            cbuf.zero_()
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            t = cbuf.cpu().numpy().reshape(n_launch, n_cta_max, TRACE_WORDS)
            t0 = t[0][t[0][:, 4] > 0][:, 0].min()
        ghz = 1.965   # SM clock under this load (cycle stamps -> microseconds)
        for k_ in range(n_launch):
            live = t[k_][t[k_][:, 4] > 0]
            cols = (live[:, [0, 10, 4]] - t0) / 1000.0
            row = {"chain_launch": k_, "kind": "boundary" if boundary else "plain", "layer": layers[k_], "ctas": int(live.shape[0]), "sms_used": int(len(set(live[:, 7].tolist()))),
                   "unit": "us from the first launch's first CTA (last repetition): median (min-max)",
                   **{name: f"{np.median(cols[:, c]):.2f} ({cols[:, c].min():.2f}-{cols[:, c].max():.2f})"
                      for c, name in enumerate(["cta_start", "wait_passed", "end"])}}
            # thread 0's cycle stamps, as microseconds after its wait passed
            names = [("reached_the_wait", 14), ("projection_loads_issued", 23), ("projection_summed", 24), ("q_arrived", 2), ("warp0_tile_landed", 3), ("warp0_scores", 16), ("warp0_probabilities", 17), ("warp0_pv", 18),
                     ("warp0_tile_done", 19), ("tiles_consumed", 8), ("partials_in_smem", 20), ("published", 9),
                     ("reduction_starts", 26), ("slot_records_first_answer", 29), ("slot_records_summed", 25), ("slot_final", 27), ("slot_phase_over", 28),
                     ("first_item_complete", 11), ("all_items_complete", 12), ("combined", 21), ("outputs_stored", 22), ("end", 13)]
            for name, slot in names:
                ok_rows = live[live[:, slot] > 0]
                if len(ok_rows):
                    d = (ok_rows[:, slot] - ok_rows[:, 1]) / ghz / 1000.0
                    row["after_wait_" + name] = f"{np.median(d):.2f} ({d.min():.2f}-{d.max():.2f})"
            if boundary:
                flags = live[:, 30]
                row["slot_records_all_there_at_first_load"] = f"{int((flags == 1).sum())} of {int((flags > 0).sum())} CTAs"
            print(json.dumps(row), flush=True)

    if wl.d_q_heads // wl.d_kv_heads <= 8:
        capture_chain()
    if 2 * (wl.d_q_heads // wl.d_kv_heads) <= 8:
        capture_chain(boundary=True)

    def capture_verify_chain(n_launch=5, reps=3):
        """Consecutive target layers replayed from one CUDA graph, one record area per launch (global-timer stamps)."""
        stride = n_cta_max * TRACE_WORDS
        cbuf = torch.zeros(n_launch * stride, dtype=torch.int64, device=dev)
        vq = r.view("vq")
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()

        def launch(l):
            r.binding.verify_attend(r.tK[l], r.tV[l], r.kv_len, vq[l], workspace=r.v_ws, out=r.v_o[l], lse=r.v_lse[l],
                                    stable_cache=True)

        with torch.cuda.stream(side):
            for l in range(n_launch):
                launch(l)
            torch.cuda.synchronize()
            binding.debug_set_trace(cbuf, stride)
            with torch.cuda.graph(g, stream=side):
                for l in range(n_launch):
                    launch(l)
            binding.debug_set_trace(None)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(reps):
            cbuf.zero_()
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
        t = cbuf.cpu().numpy().reshape(n_launch, n_cta_max, TRACE_WORDS)
        t0 = t[0][t[0][:, 4] > 0][:, 0].min()
        for k_ in range(n_launch):
            live = t[k_][t[k_][:, 4] > 0]
            cols = (live[:, [0, 10, 1, 8, 9, 3, 4]] - t0) / 1000.0
            print(json.dumps({"verify_chain_launch": k_, "ctas": int(live.shape[0]), "tiles_per_cta_min_max": [int(live[:, 6].min()), int(live[:, 6].max())],
                              "unit": "us from the first launch's first CTA: median (min-max)",
                              **{name: f"{np.median(cols[:, c]):.2f} ({cols[:, c].min():.2f}-{cols[:, c].max():.2f})"
                                 for c, name in enumerate(["cta_start", "wait_passed", "prologue_done", "softmax_loop_end",
                                                           "partial_published", "before_reduce", "end"])}}), flush=True)

    if wl.t_head_dim == 128:
        capture_verify_chain()

    L = min(3, wl.d_layers - 1)
    q1, q2 = r.view("dq0"), r.view(f"dq{r.slot_step}")
    k, v = r.view("dk0"), r.view("dv0")
    mma = [("cta_start", 0), ("prologue_done", 1), ("tiles_consumed", 2), ("partial_published", 3), ("end", 4)]
    draft = [("cta_start", 0), ("wait_passed", 10), ("end", 4)]   # the draft kernel's inner phases are cycle stamps (chain rows above)
    capture(lambda: r.mem.draft_append_attend(L, k[L], v[L], q1[L], out=r.d_o1[L], lse=r.d_lse1[L]),
            "draft_append_attend (attend_draft_kernel)", draft)
    capture(lambda: r.mem.draft_boundary_attend(L, k[L], v[L], r.view("hg")[L], r.Wk[L], r.Wv[L], r.slot_pos, q2[L],
                                                out=r.d_o2[L], lse=r.d_lse2[L]),
            "draft_boundary_attend (attend_draft_kernel + slot projection)", draft)
    vq = r.view("vq")
    LT = min(5, wl.t_layers - 1)
    tc = [("cta_start", 0), ("softmax_loop_end", 8), ("partial_published", 9), ("before_reduce", 3), ("end", 4)]
    capture(lambda: r.binding.verify_attend(r.tK[LT], r.tV[LT], r.kv_len, vq[LT], workspace=r.v_ws, out=r.v_o[LT],
                                            lse=r.v_lse[LT]),
            "verify_attend (attend_tc_kernel)" if wl.t_head_dim == 128 else "verify_attend (attend_kernel)",
            tc if wl.t_head_dim == 128 else mma)


def main():
    from paper_2608_30252_b200 import inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3_8b_32k", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--impl", default="masw", choices=["masw", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-timed-s", type=float, default=0.5,
                    help="the block of --steps steps is repeated until about this many seconds are timed (median block reported)")
    ap.add_argument("--sweep", action="store_true", help="run the prefix x batch x gamma x ratio sweep (one JSON line per point)")
    ap.add_argument("--prefill", action="store_true",
                    help="time the draft's masked prefill pass (one layer per step) instead of the decoding iteration")
    ap.add_argument("--fp8", action="store_true",
                    help="verify attention over the paged cache in bf16 and in FP8 (e4m3): us per target layer at batch 1, 4, 16")
    ap.add_argument("--loop", action="store_true",
                    help="run the packaged speculative-decoding loop on its toy models: Tok./Iter, t_d, t_t, Eq. 1")
    ap.add_argument("--timeline", action="store_true",
                    help="per-CTA phase timelines of one draft, one boundary and one verify launch (developer stamps)")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="ncu dram bytes per launch of the dominant kernel (from profiles/), echoed into the roofline")
    args = ap.parse_args()
    wl = inputs.WORKLOADS[args.workload]
    if args.sweep:
        run_sweep(args)
    elif args.fp8:
        run_fp8(args)
    elif args.loop:
        run_loop(args)
    elif args.timeline:
        run_timeline(args, wl)
    elif args.prefill:
        run_prefill(args, wl)
    elif args.impl == "reference":
        run_reference(args, wl)
    else:
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
