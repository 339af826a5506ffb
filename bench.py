#!/usr/bin/env python
"""Decode-step benchmark of the retention-eviction hot path.

A "step" is one pass of the whole hot path over one batch of synthetic input: retention gates for all
layers, append of the new token's K/V, GQA decode attention over the ragged pools, then score + global
selection + compaction (trimkv_decode_step_all).  At N = 1 the workload is the Llama-3-8B-shaped decode:
32 layers, 8 KV / 32 query heads, d 128, hidden 4096, bf16 K/V, batch 8, 32K-token context fed in
512-token chunks, budget 4096 tokens' worth (1,048,576 entries per sequence).  With N > 1 every rank holds
its own batch of sequences (independent budgets, no data-path collective): weak scaling.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
At N = 1 the line also carries `other_workloads`: the other named workloads (vision-language, multi-turn, long-context
stress) and the standalone selection sweep, each timed the same way with its own clock record.
`--gpus N` without a torchrun environment starts the N ranks itself (one process per GPU).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

_CSRC = os.path.join(ROOT, "paper_2605_09649_b200", "csrc")
ATTENTION_SOURCES = [os.path.join(_CSRC, f) for f in ("attention.cu", "mma_sync.cuh", "async_copy.cuh")]
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "attn_mma_kernel_dram_traffic.txt")


def attention_source_digest() -> str:
    h = hashlib.sha256()
    for f in ATTENTION_SOURCES:
        h.update(open(f, "rb").read())
    return h.hexdigest()


def recorded_traffic(workload: str):
    """DRAM bytes (read + write) of one launch of the dominant kernel, as an ncu capture recorded them, or None.
    Each record line is `<workload> <sha256 of the kernel's source files> <bytes per launch>`; a record counts only while
    the sources (the kernel's file and the two helper headers it is built from, concatenated) still hash to the same value,
    so a changed kernel reports no stale figure."""
    try:
        digest = attention_source_digest()
        for line in open(TRAFFIC_RECORD):
            f = line.split()
            if len(f) >= 3 and not line.startswith("#") and f[0] == workload and f[1] == digest:
                return int(f[2])
    except OSError:
        pass
    return None

METRIC = "decode tokens/s at fixed global KV budget (step time in ms_per_step, % of HBM peak in roofline)"
UNIT = "tokens/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def load_tensor_peaks():
    """Measured dense bf16 matmul rates: burst (a kernel timed alone) and sustained (inside a long run), TFLOP/s."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(p))
        return {"burst": float(d["bf16_tflops"]), "sustained": float(d["bf16_tflops_sustained"]), "kind": "measured"}
    except Exception:
        return {"burst": 1590.0, "sustained": 1400.0, "kind": "fallback"}


def algorithmic_bytes(w, entries_per_seq):
    """Bytes one decode step must move (per rank): every kept K/V row once, the per-entry retention metadata
    (lambda, c, position: 12 B) twice (histogram pass + filter pass), the gate weights once."""
    kv = w.batch * entries_per_seq * 2 * w.head_dim * (2 if w.kv_dtype == "bf16" else 4)
    meta = 2 * w.batch * entries_per_seq * 12
    gate = w.layers * (w.hidden * w.gate_hidden + w.kv_heads * w.gate_embed * w.gate_hidden + w.gate_hidden
                       + w.kv_heads * w.gate_embed) * 4
    return {"kv": kv, "meta": meta, "gate": gate, "total": kv + meta + gate}


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------------- CPU oracle arm
def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_synthetic_state(w, seed=0):
    """One sequence of the workload with its cache at the budget (M_global entries spread evenly over the pools, seeded
    N(0,1) K/V rows, seeded retention around the gate's bias) and seeded random-init gates, built on the host.
    Returns (oracle cache, generator)."""
    import numpy as np
    from oracle import trimkv_oracle as orc
    r = np.random.default_rng(seed)
    oc = orc.OracleCache(w.budget_entries, w.layers, w.kv_heads, w.q_heads, w.head_dim, w.horizon)
    per_pool = w.budget_entries // (w.layers * w.kv_heads)
    t0 = w.context
    pos = np.arange(t0 - per_pool + 1, t0 + 1, dtype=np.int64)
    for l in range(w.layers):
        for h in range(w.kv_heads):
            lam = (-np.exp(-(w.b_g + 0.05 * r.standard_normal(per_pool)))).astype(np.float32)
            oc.pos[l][h] = pos.copy()
            oc.lam[l][h] = lam
            oc.c[l][h] = orc.horizon_term_from_lambda32(lam, w.horizon)
            oc.K[l][h] = r.standard_normal((per_pool, w.head_dim))
            oc.V[l][h] = r.standard_normal((per_pool, w.head_dim))
        oc.tokens[l] = t0
    params = []
    for l in range(w.layers):
        params.append((r.standard_normal((w.gate_hidden, w.hidden)) * 0.02, np.zeros(w.gate_hidden),
                       r.standard_normal((w.kv_heads, w.gate_embed, w.gate_hidden)) * 0.02,
                       np.zeros((w.kv_heads, w.gate_embed))))
    oc.set_gate(params, r.standard_normal(w.gate_embed) * 0.02, w.b_g)
    return oc, r


def oracle_synthetic_inputs(w, r, steps):
    return [(r.standard_normal((w.layers, 1, w.hidden)), r.standard_normal((w.layers, 1, w.kv_heads, w.head_dim)),
             r.standard_normal((w.layers, 1, w.kv_heads, w.head_dim)), r.standard_normal((w.layers, w.q_heads, w.head_dim)))
            for _ in range(steps)]


def oracle_time_steps(oc, w, inputs, threads):
    """Runs the oracle, as it stands, through whole decode steps (gate, append, attention over all pools, score + full
    sort + eviction) with its library routines limited to `threads` threads.  Returns seconds per step."""
    try:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=threads)
    except Exception:
        limit = None
    times = []
    try:
        for (x, k, v, q) in inputs:
            a = time.perf_counter()
            for l in range(w.layers):
                oc.append(l, k[l], v[l], x=x[l])
                oc.decode_attention(l, q[l])
            oc.score_and_evict()
            times.append(time.perf_counter() - a)
    finally:
        if limit is not None:
            limit.restore_original_limits()
    return sum(times) / len(times)


def oracle_sample_desc(w, steps, source):
    return (f"1 of {w.batch} sequences at budget ({w.budget_entries} entries; {source}), {steps} whole decode steps "
            f"(gate+append+attention over all {w.layers * w.kv_heads} pools+score+full sort)")


def run_reference(args, w):
    from paper_2605_09649_b200 import dist_util
    rank, _, world = dist_util.env_world()
    if rank != 0:
        return                                   # under torchrun rank 0 alone runs the oracle; the others exit 0
    steps = max(1, min(args.steps, 8))
    warm = min(args.warmup, 1)
    cores = host_cores()
    oc, r = oracle_synthetic_state(w, args.seed)
    if warm:
        oracle_time_steps(oc, w, oracle_synthetic_inputs(w, r, warm), cores)
    sec = oracle_time_steps(oc, w, oracle_synthetic_inputs(w, r, steps), cores)
    value = 1.0 / sec                       # one sequence advances one token per oracle step
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded N(0,1) hidden states, K/V, random-init gates)",
        "config": {"workload": w.name, "layers": w.layers, "kv_heads": w.kv_heads, "q_heads": w.q_heads,
                   "head_dim": w.head_dim, "hidden": w.hidden, "batch_per_gpu": w.batch,
                   "budget_entries_per_seq": w.budget_entries, "context": w.context, "prefill_chunk": w.chunk, "b_g": w.b_g},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": oracle_sample_desc(w, steps, "state drawn on the host from the seed")},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def oracle_beside_gpu(cache, w, per_layer, w_g, step_inputs, first_token, seq=0):
    """The CPU baseline of the CUDA arm: the oracle on the SAME tensors.  Sequence `seq` of the GPU run is read back
    from the device (every pool: positions, fp32 retention terms, K/V rows) after the timed steps, and the oracle then
    runs whole decode steps on the GPU run's next seeded step inputs, once with one thread and once with all host
    cores.  Returns the cpu_baseline object."""
    import numpy as np
    from oracle import trimkv_oracle as orc
    f64 = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    oc = orc.OracleCache(w.budget_entries, w.layers, w.kv_heads, w.q_heads, w.head_dim, w.horizon)
    lens = cache.lengths()[seq]
    cap = int(lens.max()) + 1
    for l in range(w.layers):
        for h in range(w.kv_heads):
            pos, lam, c, k, v = cache.pool(seq, l, h, cap, with_kv=True)
            order = np.argsort(pos.numpy(), kind="stable")
            oc.pos[l][h] = pos.numpy().astype(np.int64)[order]
            oc.lam[l][h] = lam.numpy()[order]
            oc.c[l][h] = c.numpy()[order]
            oc.K[l][h] = f64(k)[order]
            oc.V[l][h] = f64(v)[order]
        oc.tokens[l] = first_token
    oc.set_gate([tuple(f64(t) for t in p) for p in per_layer], f64(w_g), w.b_g)
    big = w.budget_entries > 100000
    n1, nc = (2, 3) if big else (4, 8)
    ins = []
    for i in range(n1 + nc):
        X, Kt, Vt, Q = step_inputs(i)
        ins.append((f64(X[:, seq])[:, None], f64(Kt[:, seq])[:, None], f64(Vt[:, seq])[:, None], f64(Q[:, seq])))
    cores = host_cores()
    sec1 = oracle_time_steps(oc, w, ins[:n1], 1)
    secc = oracle_time_steps(oc, w, ins[n1:], cores)
    return {"value": 1.0 / secc, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": oracle_sample_desc(w, nc, f"sequence {seq} of the GPU run read back from the device, then the GPU run's "
                                                "next seeded step inputs"),
            "one_thread": {"value": 1.0 / sec1, "unit": UNIT, "cores": 1, "steps": n1}}


# ------------------------------------------------------------------------------------------------- CUDA arm
def measure_workload(args, w, K, W, rank, world, local_rank, main):
    """Builds the workload's cache on this rank's GPU (chunked prefill with evictions, earlier turns of a dialogue), then
    times K whole decode steps after W warm-up steps (device-resident inputs; CUDA events; barrier on both sides), the
    per-phase times with the phases serialised, and the end-to-end form with host buffers.  main: the headline
    workload (per-phase detail, CPU baseline); otherwise a compact record is enough."""
    import torch
    from paper_2605_09649_b200 import binding, dist_util, workloads

    dev = f"cuda:{local_rank}"
    # weak scaling: the job holds world x batch independent sequences; this rank owns a contiguous block of them
    seq_lo, seq_hi = workloads.shard_sequences(world * w.batch, rank, world)
    seed = args.seed + 1000 * (seq_lo // w.batch)       # every rank draws different sequences

    per_pool = w.budget_entries // (w.layers * w.kv_heads) if args.fixed_budget else 0
    cache = binding.TrimKV.from_workload(w, retention_bias=args.retention_bias, per_pool_budget=per_pool)
    per_layer, w_g = workloads.gate_params(w, seed, device=dev)
    if args.skew > 0:
        # per-(layer, head) logit offsets through b2 (b2 . w_g shifts s): retention then differs strongly between heads and
        # the pools become ragged, as the paper reports for trained gates; the default run keeps the plain random init
        off = workloads.head_logit_offsets(w, seed, args.skew, device=dev)
        wn = w_g / (w_g * w_g).sum()
        per_layer = [(W1, b1, W2, (b2 + off[l][:, None] * wn[None, :]).contiguous()) for l, (W1, b1, W2, b2) in enumerate(per_layer)]
    for l, p in enumerate(per_layer):
        cache.set_gate(l, *p)
    cache.set_shared_projection(w_g, w.b_g)
    bank = workloads.ProjectionBank(w, seed, device=dev)

    # ---- untimed: chunked prefill with eviction after every chunk (library time measured with events on the side)
    def prefill(start, count):
        """Appends tokens [start, start + count) in chunks with an eviction after each; returns (ms of library work, chunks)."""
        ms, chunks, done = 0.0, 0, 0
        while done < count:
            n = min(w.chunk, count - done)
            evs, aevs = [], []
            n_old = cache.lengths().to(torch.float64) if args.prefill_attention else None     # [B, L, H] before the chunk
            for l in range(w.layers):
                x = workloads.hidden_states(w, seed, l, start + done, n, device=dev)
                qc, k, v = workloads.project_qkv(w, bank, l, x)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                cache.append(l, k, v, x=x)
                if args.prefill_attention:
                    a2, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a2.record()
                    cache.prefill_attention(l, qc)
                    b2.record()
                    aevs.append((a2, b2))
                if l == w.layers - 1:
                    cache.score_and_evict()
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            ms += sum(a.elapsed_time(b) for a, b in evs)
            if aevs:
                # causal work of this chunk: query head (b, j, hq) sees n_old + j + 1 entries of its pool, 4 d flops each
                fl = 4.0 * w.head_dim * (w.q_heads // w.kv_heads) * (n * n_old.sum().item() + n_old.numel() * n * (n + 1) / 2)
                attn_stats["ms"] += sum(a.elapsed_time(b) for a, b in aevs)
                attn_stats["flops"] += fl
                attn_stats["last_ms"] = sum(a.elapsed_time(b) for a, b in aevs)
                attn_stats["last_flops"] = fl
            chunks += 1
            done += n
        return ms, chunks

    attn_stats = {"ms": 0.0, "flops": 0.0, "last_ms": 0.0, "last_flops": 0.0}
    t_setup = time.time()
    tokens_seen = 0
    prefill_ms, prefill_chunks, early_decode_ms, early_decode_steps = 0.0, 0, 0.0, 0
    for turn in range(w.turns):
        ms, ch = prefill(tokens_seen, w.context)
        prefill_ms += ms; prefill_chunks += ch
        tokens_seen += w.context
        if turn < w.turns - 1:
            # earlier turns of a dialogue: their decode steps run here (timed coarsely); the last turn's are the timed region
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            sets = []
            for i in range(4):
                xs, ks, vs, qs = [], [], [], []
                for l in range(w.layers):
                    x = workloads.hidden_states(w, seed, l, tokens_seen + i, 1, device=dev)
                    q, k, v = workloads.project_qkv(w, bank, l, x)
                    xs.append(x[:, 0]); ks.append(k[:, 0]); vs.append(v[:, 0]); qs.append(q[:, 0])
                sets.append([torch.stack(t).contiguous() for t in (xs, ks, vs, qs)])
            o = torch.empty_like(sets[0][3])
            a.record()
            for i in range(w.decode_steps):
                X, Kt, Vt, Q = sets[i % 4]
                cache.decode_step_all(Kt, Vt, Q, o, x=X)
            b.record()
            torch.cuda.synchronize()
            early_decode_ms += a.elapsed_time(b); early_decode_steps += w.decode_steps
            tokens_seen += w.decode_steps
    cache.sync_status()
    entries = int(cache.lengths()[0].sum())
    t_setup = time.time() - t_setup

    # ---- per-step inputs, resident in HBM before the timed region
    def step_inputs(i):
        xs, ks, vs, qs = [], [], [], []
        for l in range(w.layers):
            x = workloads.hidden_states(w, seed, l, tokens_seen + i, 1, device=dev)
            q, k, v = workloads.project_qkv(w, bank, l, x)
            xs.append(x[:, 0]); ks.append(k[:, 0]); vs.append(v[:, 0]); qs.append(q[:, 0])
        return [torch.stack(t).contiguous() for t in (xs, ks, vs, qs)]

    NSETS = min(16, W + K)                       # distinct input sets, used round robin (each 8 MB at the llama shape)
    inputs = [step_inputs(i) for i in range(NSETS)]
    out = torch.empty_like(inputs[0][3])
    torch.cuda.synchronize()

    done_steps = [0]                             # decode steps this cache has taken since the prefill

    def step(i):
        X, Kt, Vt, Q = inputs[i % NSETS]
        cache.decode_step_all(Kt, Vt, Q, out, x=X)
        done_steps[0] += 1

    # the decode loop runs on the handle's own highest-priority stream (a serving loop would do the same): the step's
    # attention chain then needs no hand-off from and to the caller's stream
    torch.cuda.synchronize()
    loop_stream = cache.step_stream()
    torch.cuda.set_stream(loop_stream)
    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    dist_util.barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = binding.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cache.profile(2)          # two events per step around the attention kernel, on the stream it is launched on
    torch.cuda.synchronize()
    e0.record()
    for i in range(K):
        step(W + i)
    e1.record()
    torch.cuda.synchronize()
    dist_util.barrier()
    launches = binding.kernel_launches() - launches0
    ms_total = e0.elapsed_time(e1)
    live = cache.profile_read()["attn_main"]
    cache.profile(False)
    if rank == 0:                            # a short timed region: keep the GPU under the same load until nvidia-smi has sampled it
        t_load = time.perf_counter()
        while K * ms_total / max(K, 1) < 600.0 and time.perf_counter() - t_load < 0.6 - ms_total * 1e-3:
            for i in range(16):
                step(W + K + i)
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    cache.sync_status()
    ms_step = dist_util.max_over_ranks(ms_total / K, device=dev)
    tokens_per_step = dist_util.sum_over_ranks(w.batch, device=dev)
    value = tokens_per_step / (ms_step * 1e-3)

    # ---- per-phase device time over more steps with the phases run back to back on one stream (no overlap), CUDA
    # events around each phase: what each kernel takes when it has the memory system to itself
    KP = min(K, 32)
    cache.set_overlap(False)
    cache.profile(True)
    for i in range(KP):
        step(W + K + i)
    phases = cache.profile_read()
    cache.profile(False)
    cache.set_overlap(True)

    # ---- end to end: host buffers in, host result out, copies inside the timed region
    KE = min(K, 32)
    host_in = [[t.cpu().pin_memory() for t in inputs[i % NSETS]] for i in range(min(KE, NSETS))]
    host_out = torch.empty_like(out, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_in[0])
    d2h = host_out.numel() * host_out.element_size()

    def e2e_loop(n):
        for i in range(n):
            hX, hK, hV, hQ = host_in[i % len(host_in)]
            cache.decode_step_all_host(hK, hV, hQ, host_out, x=hX)   # the C-ABI call with host buffers: copies inside
            torch.cuda.current_stream().synchronize()         # the caller needs the step's result before the next token
            done_steps[0] += 1

    e2e_loop(2)
    torch.cuda.synchronize()
    dist_util.barrier()
    e0.record()
    e2e_loop(KE)
    e1.record()
    torch.cuda.synchronize()
    dist_util.barrier()
    e2e_ms = dist_util.max_over_ranks(e0.elapsed_time(e1) / KE, device=dev)
    e2e_value = tokens_per_step / (e2e_ms * 1e-3)
    # where the end-to-end step's time goes: the same loop with events around the copies and the kernels (the events
    # themselves cost a little, so this loop is not the one that is reported as the end-to-end number)
    cache.profile(True)
    t0 = time.perf_counter()
    e2e_loop(KE)
    torch.cuda.synchronize()
    wall_prof = (time.perf_counter() - t0) / KE * 1e3
    eph = cache.profile_read()
    cache.profile(False)
    per = lambda name: eph[name][0] / max(eph[name][1], 1)
    breakdown = {"h2d_kvq_ms": per("h2d_kvq"), "h2d_x_ms": per("h2d_x"), "append_ms": per("append"), "attention_ms": per("attn_main"),
                 "gate_ms": per("gate"), "select_ms": per("select"), "compact_ms": per("compact"), "d2h_out_ms": per("d2h_out"),
                 "what": "device time of each part of trimkv_decode_step_all_host (gate, x copy and selection run beside the "
                         "attention kernel); critical path = h2d_kvq + append + attention + compact + d2h_out; the rest of "
                         "ms_per_step is host launch and synchronisation latency.  q and the output sit in pinned host memory "
                         "and are read / written there by the attention kernel itself (no copy is queued: their bytes cross "
                         "the bus inside attention_ms); K and V are copied by copy engine (h2d_kvq), or read in place by the "
                         "append kernel when they are under 512 KB together"}
    breakdown["critical_path_ms"] = sum(breakdown[k] for k in ("h2d_kvq_ms", "append_ms", "attention_ms", "compact_ms", "d2h_out_ms"))
    breakdown["host_latency_ms"] = max(0.0, e2e_ms - breakdown["critical_path_ms"])
    breakdown["wall_ms_per_step_with_events"] = wall_prof
    cache.sync_status()
    lens = cache.lengths()
    assert int(lens[0].sum()) == min(w.budget_entries, entries), "budget invariant violated"
    assert per_pool == 0 or int(lens.max()) <= per_pool

    modality = None
    if w.visual_period > 0 and rank == 0:
        # what the global budget kept of each modality (sequence 0): a token's modality follows from its position and
        # the workload's layout; the cache itself stores no modality tag
        pos = torch.cat([cache.kept(0, l, h, int(lens[0, l, h]) + 1) for l in range(w.layers) for h in range(w.kv_heads)])
        vis = workloads.is_visual(w, pos.to(torch.int64) - 1)
        prompt = workloads.is_visual(w, torch.arange(tokens_seen + done_steps[0]))
        modality = {"kept_entries": int(pos.numel()), "kept_visual_entries": int(vis.sum()),
                    "kept_visual_share": float(vis.float().mean()), "visual_share_of_tokens_seen": float(prompt.float().mean())}
    peak, peak_kind = load_peaks()
    ab = algorithmic_bytes(w, entries + w.layers * w.kv_heads)
    if args.retention_bias:                                        # lambda and position of every entry ride along
        extra_b = w.batch * (entries + w.layers * w.kv_heads) * 8
        ab["kv"] += extra_b; ab["total"] += extra_b
    attn_ms_per = live[0] / max(live[1], 1)                       # timed region: beside the gate and the selection
    achieved = ab["kv"] / (attn_ms_per * 1e-3) / 1e9 if attn_ms_per > 0 else 0.0
    iso_ms = phases["attn_main"][0] / max(phases["attn_main"][1], 1)
    iso_gbs = ab["kv"] / (iso_ms * 1e-3) / 1e9 if iso_ms > 0 else 0.0
    step_gbs = ab["total"] / (ms_step * 1e-3) / 1e9
    res = {"w": w, "K": K, "W": W, "value": value, "ms_step": ms_step, "launches": launches, "clocks": clocks, "entries": entries,
           "lens_min_max": [int(lens[0].min()), int(lens[0].max())], "t_setup": t_setup, "tokens_seen": tokens_seen,
           "prefill_ms": prefill_ms, "prefill_chunks": prefill_chunks, "attn_stats": attn_stats,
           "early_decode": early_decode_ms / early_decode_steps if early_decode_steps else None,
           "ab": ab, "attn_ms_per": attn_ms_per, "achieved": achieved, "iso_ms": iso_ms, "iso_gbs": iso_gbs, "step_gbs": step_gbs,
           "phases": {k: v[0] / KP for k, v in phases.items() if v[1]}, "peak": peak, "peak_kind": peak_kind,
           "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "steps": KE, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "breakdown": breakdown},
           "per_pool": per_pool, "seqs": [seq_lo, seq_hi], "cpu": None, "modality": modality}
    if main and rank == 0 and not args.no_cpu_baseline:
        res["cpu"] = oracle_beside_gpu(cache, w, per_layer, w_g, lambda i: step_inputs(done_steps[0] + i),
                                       tokens_seen + done_steps[0])
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())
    cache.close()
    del cache, inputs, host_in
    torch.cuda.empty_cache()
    return res


def run_ours(args, w):
    import torch
    from paper_2605_09649_b200 import dist_util

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local_rank, world = dist_util.init("nccl") if int(os.environ.get("WORLD_SIZE", "1")) > 1 else (0, 0, 1)
    if local_rank >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank} needs CUDA device {local_rank}; {torch.cuda.device_count()} present")
    torch.cuda.set_device(local_rank)
    K, W = args.steps, args.warmup
    r = measure_workload(args, w, K, W, rank, world, local_rank, main=True)
    if rank != 0:
        return
    tpk = load_tensor_peaks()
    ab, peak, peak_kind, attn_stats = r["ab"], r["peak"], r["peak_kind"], r["attn_stats"]
    default_config = args.skew == 0 and args.context is None and args.layers is None and not args.retention_bias
    line = {
        "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": r["ms_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.kv_dtype == "bf16" else "f32",
        "data": "synthetic (seeded N(0,1) hidden states; K/V/Q from random-init projections; random-init gates)",
        "config": {"workload": w.name, "layers": w.layers, "kv_heads": w.kv_heads, "q_heads": w.q_heads,
                   "head_dim": w.head_dim, "hidden": w.hidden, "batch_per_gpu": w.batch,
                   "budget_entries_per_seq": w.budget_entries, "context": w.context, "prefill_chunk": w.chunk,
                   "entries_per_seq_during_step": r["entries"] + w.layers * w.kv_heads, "b_g": w.b_g, "skew": args.skew, "retention_bias": bool(args.retention_bias), "fixed_per_pool_budget": r["per_pool"],
                   "pool_len_min_max": r["lens_min_max"],
                   "parallelism": f"{world * w.batch} independent sequences sharded over {world} rank(s) (rank 0: {r['seqs']}), no collective",
                   "l2": "inputs larger than L2 (each step streams the whole cache)", "setup_s": round(r["t_setup"], 1),
                   "turns": w.turns, "tokens_before_timed_region": r["tokens_seen"],
                   "prefill": {"chunks": r["prefill_chunks"], "ms_per_chunk": r["prefill_ms"] / max(r["prefill_chunks"], 1),
                               "tokens_per_s": w.batch * w.chunk / (r["prefill_ms"] / max(r["prefill_chunks"], 1) * 1e-3) if r["prefill_ms"] > 0 else None,
                               "what": "gate + append of every layer and one eviction per chunk" +
                                       (", with the chunk's causal attention" if args.prefill_attention else " (no chunk attention)"),
                               "chunk_attention": None if not args.prefill_attention else {
                                   "kernel": "prefill_attn_tc_kernel (tcgen05) where the shapes allow, else mma.sync",
                                   "last_chunk_ms_all_layers": attn_stats["last_ms"],
                                   "last_chunk_tflops": attn_stats["last_flops"] / (attn_stats["last_ms"] * 1e-3) / 1e12 if attn_stats["last_ms"] > 0 else None,
                                   "bound": "tensor", "peak_tflops_burst": tpk["burst"], "peak_tflops_sustained": tpk["sustained"],
                                   "peak_kind": f"of {tpk['kind']}",
                                   "frac_of_burst": (attn_stats["last_flops"] / (attn_stats["last_ms"] * 1e-3) / 1e12 / tpk["burst"])
                                                    if attn_stats["last_ms"] > 0 else None,
                                   "frac_of_sustained": (attn_stats["last_flops"] / (attn_stats["last_ms"] * 1e-3) / 1e12 / tpk["sustained"])
                                                        if attn_stats["last_ms"] > 0 else None,
                                   "flops": "causal: 4 d per (query head, visible entry); masked tile parts not counted"}},
                   "earlier_turn_decode_ms_per_step": r["early_decode"], "kept_by_modality": r["modality"]},
        "roofline": {"bound": "hbm", "kernel": "attn_mma_kernel", "achieved": r["achieved"], "peak": peak, "unit": "GB/s",
                     "frac": r["achieved"] / peak, "peak_kind": f"of {peak_kind} (a copy's read + write rate: a read-only stream can exceed it)",
                     "traffic": recorded_traffic(w.name) if default_config else None,
                     "traffic_source": "ncu capture recorded under profiles/, valid while the kernel's source hashes to the recorded value",
                     "algorithmic_bytes_per_launch": ab["kv"], "avg_launch_ms": r["attn_ms_per"],
                     "note": "timed region: the kernel shares HBM with the gate and selection kernels running beside it",
                     "alone": {"avg_launch_ms": r["iso_ms"], "achieved": r["iso_gbs"], "frac": r["iso_gbs"] / peak},
                     "step": {"algorithmic_bytes": ab, "achieved_gbs": r["step_gbs"], "frac_of_peak": r["step_gbs"] / peak,
                              "frac_of_8tbs_nominal": r["step_gbs"] / 8000.0},
                     "phase_ms_per_step_serial": r["phases"]},
        "cpu_baseline": r["cpu"],
        "e2e": r["e2e"],
        "gpu_launches": r["launches"],
        "clocks": r["clocks"],
    }
    if world == 1 and args.workload == "llama8b_32k" and default_config and not args.no_other_workloads:
        line["other_workloads"] = other_workloads(args)
    print(json.dumps(line), flush=True)


def other_workloads(args):
    """The other named workloads at their full shapes and the standalone selection sweep, each timed like the headline
    workload (device-resident inputs, CUDA events, its own clock record): compact records for the one JSON line."""
    import copy
    from paper_2605_09649_b200 import workloads
    out = {}
    # the last entry is the headline shape with strongly different retention per (layer, head): ragged pools (0 .. 32K
    # entries), as the paper reports for trained gates; the plain random init of the headline run gives equal pools
    for name, skew in (("qwen_vl_16k", 0.0), ("stress_128k", 0.0), ("multiturn", 0.0), ("llama8b_32k", 3.0)):
        w = workloads.WORKLOADS[name]
        a2 = copy.copy(args)
        a2.skew = skew
        r = measure_workload(a2, w, 32, 3, 0, 1, 0, main=False)
        name = name if skew == 0 else f"{name}_skew{skew:g}"
        out[name] = {"ms_per_step": r["ms_step"], "tokens_per_s": r["value"], "steps": r["K"], "warmup": r["W"],
                     "batch": w.batch, "skew": skew, "pool_len_min_max": r["lens_min_max"], "entries_per_seq_during_step": r["entries"] + w.layers * w.kv_heads,
                     "algorithmic_bytes": r["ab"], "step_gbs": r["step_gbs"], "frac_of_measured_hbm": r["step_gbs"] / r["peak"],
                     "frac_of_8tbs_nominal": r["step_gbs"] / 8000.0,
                     "attention_kernel": {"avg_launch_ms": r["attn_ms_per"], "achieved_gbs": r["achieved"], "frac": r["achieved"] / r["peak"]},
                     "e2e_ms_per_step": r["e2e"]["ms_per_step"], "e2e_tokens_per_s": r["e2e"]["value"],
                     "gpu_launches": r["launches"], "clocks": r["clocks"], "setup_s": round(r["t_setup"], 1),
                     "earlier_turn_decode_ms_per_step": r["early_decode"]}
        if r["modality"]:
            out[name]["kept_by_modality"] = r["modality"]
    rows, clocks = select_sweep_rows(args, (20, 24, 28), 5, 3)
    out["select_sweep"] = {"rows": rows, "clocks": clocks, "l2": "flushed between timed calls",
                           "what": "trimkv_select_topk over n fp32 scores uniform in [-8, 0]; gbs counts one pass of 4 n bytes per call"}
    return out


# ------------------------------------------------------------------------------------------------- selection sweep
def select_sweep_rows(args, exps, K, W):
    """Times trimkv_select_topk over flat fp32 score arrays (uniform in [-8, 0]) of 2^p scores for p in exps, k in
    {n/8, n/2, n - 512}: median of K calls after W warm-up calls, L2 flushed before each timed call.  Returns
    (rows, clock record)."""
    import numpy as np
    import torch
    from paper_2605_09649_b200 import binding, workloads
    dev = f"cuda:{torch.cuda.current_device()}"
    peak, _ = load_peaks()
    flush = torch.empty(192 << 20, dtype=torch.uint8, device=dev)            # larger than L2
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    rows = []
    for p in exps:
        n = 1 << p
        s = workloads.selection_scores(n, seed=args.seed, device=dev)
        bits = torch.empty((n + 63) // 64, dtype=torch.int64, device=dev)
        ws = torch.empty(binding.select_workspace_bytes(n), dtype=torch.uint8, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        for k in (n // 8, n // 2, n - 512):
            for _ in range(W):
                binding.select_topk(s, k, bits, ws, status)
            ms = []
            launches0 = binding.kernel_launches()
            for _ in range(K):
                flush.zero_()                                                 # L2 flush between timed calls
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                binding.select_topk(s, k, bits, ws, status)
                e1.record()
                torch.cuda.synchronize()
                ms.append(e0.elapsed_time(e1))
            assert int(status.item()) == 0
            m = float(np.median(ms))
            gbs = 4.0 * n / (m * 1e-3) / 1e9
            rows.append({"n": n, "k_keep": k, "ms": m, "gbs": gbs, "frac_of_measured_hbm": gbs / peak,
                         "launches_per_call": (binding.kernel_launches() - launches0) // K})
        del s, bits, ws
    torch.cuda.synchronize()
    return rows, sampler.stop()


def run_select_sweep(args):
    """Standalone global selection, N = 2^sweep_min .. 2^sweep_max, timed alone.  One JSON line."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the selection has no CPU fallback")
    torch.cuda.set_device(0)
    peak, peak_kind = load_peaks()
    K, W = min(max(args.steps, 1), 10), max(args.warmup, 3)
    rows, clocks = select_sweep_rows(args, range(args.sweep_min, args.sweep_max + 1), K, W)
    best = max(r["gbs"] for r in rows if r["n"] == rows[-1]["n"])
    line = {"metric": "standalone global selection, GB/s of score bytes per call", "unit": "GB/s", "value": best, "n_gpus": 1,
            "steps": K, "warmup": W, "higher_is_better": True, "dtype": "f32", "data": "synthetic (uniform log-retention in [-8, 0])",
            "config": {"workload": "select_sweep", "n": [1 << args.sweep_min, 1 << args.sweep_max], "l2": "flushed between timed calls"},
            "roofline": {"bound": "hbm", "kernel": "flat selection (whole call)", "achieved": best, "peak": peak, "unit": "GB/s",
                         "frac": best / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                         "note": "achieved counts ONE pass of 4 N bytes per call"},
            "sweep": rows, "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_sharded_stages(args):
    """Layer-sharded eviction round (one sequence's layers over several GPUs, one global budget): device time of every
    rank-local stage and the bytes each exchange moves, measured on ONE GPU with the ranks emulated as threads of this
    process, each with a handle holding its slice of the layers and a stream of its own.  The ranks meet on the host
    between stages (no kernel waits for another rank's kernel), and the exchanges are plain tensor stacks, so this says
    what the stages cost and how small the exchanges are, not what a multi-GPU run takes.  One JSON line."""
    import threading
    import torch
    from paper_2605_09649_b200 import binding, sharded, workloads
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the stages have no CPU fallback")
    torch.cuda.set_device(0)
    dev = "cuda"
    w = workloads.WORKLOADS[args.workload]
    world = args.emulated_ranks
    if w.layers % world:
        raise SystemExit("--emulated-ranks must divide the number of layers")
    per, LH = w.layers // world, w.layers * w.kv_heads
    rounds, warm = max(args.steps, 1), max(args.warmup, 3)
    context = args.context if args.context is not None else (w.budget_entries // LH + 2 * w.chunk)
    slots, barrier = [None] * world, threading.Barrier(world)

    class Comm:                                           # all ranks live in this process: gather = stack
        def __init__(self, rank):
            self.rank, self.world, self.bytes = rank, world, {}

        def all_gather(self, t, what="gather"):
            slots[self.rank] = t
            torch.cuda.current_stream().synchronize()
            barrier.wait()
            out = torch.stack(list(slots))
            torch.cuda.current_stream().synchronize()     # the other ranks' tensors have been read before they move on
            barrier.wait()
            self.bytes[what] = self.bytes.get(what, 0) + t.numel() * t.element_size() * (world - 1)
            return out

        def all_reduce_sum(self, t):
            g = self.all_gather(t.clone(), "reduce")
            t.copy_(g.sum(0).to(t.dtype))
            return t

    class Timed(sharded.CudaStages):                      # CUDA events around every stage call, on the rank's stream
        def __init__(self, cache):
            super().__init__(cache)
            self.on, self.ev = False, []

    def timed(name):
        plain = getattr(sharded.CudaStages, name)

        def call(self, *a, **k):
            if not self.on:
                return plain(self, *a, **k)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            r = plain(self, *a, **k)
            e1.record()
            self.ev.append((name, e0, e1))
            return r
        return call
    for name in ("sample", "bracket", "filter", "candidates", "resolve", "compact"):
        setattr(Timed, name, timed(name))

    results, errors = [None] * world, []

    def rank_body(rank):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                cache = binding.TrimKV.from_workload(w.replace(layers=per), shard_total_layers=w.layers, shard_layer0=rank * per)
                stages, comm = Timed(cache), Comm(rank)
                gen = torch.Generator(device=dev)
                gen.manual_seed(args.seed * 1000 + rank)
                held, cands = 0, []

                def one_round(n):
                    nonlocal held
                    kv = torch.zeros(w.batch, n, w.kv_heads, w.head_dim, device=dev, dtype=workloads.torch_dtype(w.kv_dtype))
                    for l in range(per):
                        lam = -torch.rand(w.batch, n, w.kv_heads, device=dev, generator=gen) * 0.05
                        cache.append(l, kv, kv, lam=lam)
                    n_total = held + n * LH
                    if n_total > w.budget_entries:
                        info = sharded.sharded_evict(stages, comm, n_total, n_total - w.budget_entries)
                        held = w.budget_entries
                        return info
                    held = n_total
                    return None

                for off in range(0, context, w.chunk):
                    one_round(w.chunk)
                for _ in range(warm):
                    one_round(1)
                stages.on, comm.bytes = True, {}
                for _ in range(rounds):
                    info = one_round(1)
                    cands.append(info["candidates"])
                    assert not info["fallback"]
                torch.cuda.synchronize()
                per_stage = {}
                for name, e0, e1 in stages.ev:
                    per_stage.setdefault(name, []).append(e0.elapsed_time(e1))
                results[rank] = ({k: sum(v) / len(v) for k, v in per_stage.items()}, dict(comm.bytes), sum(cands) / len(cands))
                cache.check_invariants()
                cache.close()
        except BaseException as e:                        # noqa: BLE001
            errors.append(e)
            barrier.abort()

    threads = [threading.Thread(target=rank_body, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    real = [e for e in errors if not isinstance(e, threading.BrokenBarrierError)]
    if errors:
        raise (real[0] if real else errors[0])
    stage_ms = {k: max(r[0][k] for r in results) for k in results[0][0]}
    line = {"metric": "layer-sharded eviction round: ms per rank-local stage call on the rank's stream (max over emulated ranks)", "unit": "ms",
            "value": sum(stage_ms.values()), "n_gpus": 1, "emulated_ranks": world, "steps": rounds, "warmup": warm,
            "higher_is_better": False, "dtype": "int64", "data": "synthetic (uniform log-retention, zero K/V)",
            "config": {"workload": w.name, "layers_per_rank": per, "budget_entries": w.budget_entries, "batch": w.batch,
                       "round": "one decode step: 1 token appended to every layer, then the eviction round"},
            "stage_ms": stage_ms,
            "exchange_bytes_received_per_rank_and_round": {k: v / rounds for k, v in results[0][1].items()},
            "candidates_per_round": results[0][2],
            "note": "ranks emulated as threads on one GPU: their kernels share it, and the events around a stage call also "
                    "span the time the host needs to queue its kernels (two Python threads, one interpreter), so a stage's "
                    "figure is an upper bound of what a rank alone would take: the kernels themselves are in the launch list "
                    "under profiles/; the exchanges are tensor stacks here (NCCL all-gather / all-reduce between GPUs)"}
    print(json.dumps(line), flush=True)


def spawn_ranks(args):
    """`--gpus N` outside a torchrun environment: start the N ranks here, one process per GPU (torch.distributed.run on
    this node, rendezvous on 127.0.0.1).  Returns the launcher's exit code."""
    import socket
    import torch
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    if have < args.gpus:
        sys.stderr.write(f"bench.py --gpus {args.gpus}: needs {args.gpus} CUDA devices, found {have}\n")
        return 2
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")                   # the communicator's set-up lines, on stderr: stdout carries the JSON line
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env, cwd=ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_32k")
    ap.add_argument("--context", type=int, default=None, help="override the prompt length (development only)")
    ap.add_argument("--b-g", type=float, default=None, help="override the shared gate bias")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--skew", type=float, default=0.0, help="std of per-(layer, head) gate-logit offsets (ragged pools)")
    ap.add_argument("--retention-bias", action="store_true",
                    help="decode attention with the retention-gated weights of Sec. 2.2 (reads 8 more bytes per entry)")
    ap.add_argument("--fixed-budget", action="store_true",
                    help="the fixed per-head budget variant (every pool keeps budget / (layers * kv_heads) entries)")
    ap.add_argument("--prefill-attention", action="store_true",
                    help="also run the chunk's causal attention over the cache during the (untimed) prefill and report it")
    ap.add_argument("--layers", type=int, default=None,
                    help="override the layer count, budget scaled with it (development and small profiling captures only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="leave out the other named workloads and the selection sweep (they add about half a minute)")
    ap.add_argument("--select-sweep", action="store_true", help="time the standalone selection over 2^20..2^28 scores instead")
    ap.add_argument("--sharded-stages", action="store_true",
                    help="time the rank-local stages of the layer-sharded eviction round with ranks emulated on one GPU instead")
    ap.add_argument("--emulated-ranks", type=int, default=2)
    ap.add_argument("--sweep-max", type=int, default=28)
    ap.add_argument("--sweep-min", type=int, default=20)
    args = ap.parse_args()
    if args.select_sweep:
        return run_select_sweep(args)
    if args.sharded_stages:
        return run_sharded_stages(args)
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    in_torchrun = "WORLD_SIZE" in os.environ and "RANK" in os.environ
    if in_torchrun and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={os.environ['WORLD_SIZE']}")
    if args.impl == "ours" and args.gpus > 1 and not in_torchrun:
        sys.exit(spawn_ranks(args))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2605_09649_b200 import workloads
    w = workloads.WORKLOADS[args.workload]
    if args.context is not None:
        w = w.replace(context=args.context)
    if args.b_g is not None:
        w = w.replace(b_g=args.b_g)
    if args.layers is not None:                       # a shallower model of the same shapes (small profiling captures)
        w = w.replace(layers=args.layers, budget_entries=w.budget_entries // w.layers * args.layers)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
