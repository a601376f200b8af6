#!/usr/bin/env python
"""Benchmark of SANTA++ decode attention on B200.

One "step" is one decode token through `--layers` independently seeded layers of the
Qwen2.5-7B single-layer workload (batch 1, 28 query heads over 4 KV heads, head_dim 128,
32K-token prompt, suffix growing to 256, parents of 512 with 32 representatives, 32 sampled
teams): per layer, the whole hot path (representative scoring, Gumbel-top-K sampling, read
plan, exact attention over the sampled teams and the suffix, split-K merge). The layers are
visited round-robin so that every layer-step reads K/V from HBM, not from L2 (28 layers hold
1.8 GiB of packed K/V against 126 MB of L2).

Prints ONE JSON line (rank 0). `value` is microseconds per layer-step with all inputs resident
in HBM, replayed from CUDA graphs; `e2e` is the same through host buffers (pinned host to
device copies of the step's queries, new suffix rows and counters, device to host read of the
outputs, inside the timed region). With the default workload the line also carries `batched`:
the same measurement on the ragged 32-sequence batch (two layers, 30 steps), the size at which
the operator is bandwidth-bound rather than latency-bound (`--no-batched` skips it), `mid_batch` and
`long_context` (configs 3 and 5), `shared_latent` (rows of 512 + 64 values shared by 16 heads, 32
sequences of 8K, `--workload latent_8k` on its own) and `kmeans_parents`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--layers L]
"""
import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attn_us_per_layer_step"
UNIT = "us"
N_STEP_INPUTS = 8          # distinct (query, suffix length, step) inputs cycled through

# DRAM bytes (read + write) of one attend_kernel launch, recorded from an ncu capture of this
# kernel on the same per-launch work (default seed, independent keys, contiguous parents). A
# recorded figure, not one measured by this run: it is reported as `traffic` together with
# `traffic_kind`, and left out (null) for any other variant of the workload.
NCU_TRAFFIC_BYTES = {
    "qwen7b_b1_32k": 34.57e6,
    "qwen7b_b8_32k": 405.3e6,
    "ragged": 1037.1e6,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=28)
    ap.add_argument("--workload", default="qwen7b_b1_32k",
                    choices=["qwen7b_b1_32k", "qwen7b_b8_32k", "ragged", "long_128k", "paper_point_32k", "small_gqa", "latent_8k"])
    ap.add_argument("--n-sample", type=int, default=0, help="override K")
    ap.add_argument("--latent-seqs", type=int, default=32, help="sequences of the latent_8k workload")
    ap.add_argument("--key-layout", default="iid", choices=["iid", "runs"],
                    help="cluster of each prompt row: independent draws, or geometric runs (positional locality)")
    ap.add_argument("--elem", default="bf16", choices=["bf16", "fp16"], help="16-bit element type of q, K, V")
    ap.add_argument("--parents", default="contiguous", choices=["contiguous", "centres", "kmeans"],
                    help="contiguous: Algorithm 4; kmeans: Algorithm 3 with the paper's settings (fit on the GPU); "
                         "centres: Algorithm 3 without the fit, on the first of the centres the synthetic keys were "
                         "drawn around (uneven parents; not a model of a converged fit)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-stages", action="store_true")
    ap.add_argument("--no-batched", action="store_true", help="skip the extra bandwidth-bound workload")
    return ap.parse_args()


def make_spec(args, seed):
    from paper_2609_35629_b200 import synth
    if args.workload == "qwen7b_b1_32k":
        spec = synth.spec_qwen_b1(seed=seed)
    elif args.workload == "qwen7b_b8_32k":
        spec = synth.spec_qwen_b8(seed=seed)
    elif args.workload == "ragged":
        spec = synth.spec_ragged(seed=seed)
    elif args.workload == "long_128k":
        spec = synth.spec_long(seed=seed)
    elif args.workload == "paper_point_32k":
        spec = synth.spec_paper_point(seed=seed)
    else:
        spec = synth.spec_small_gqa(seed=seed)
    if args.n_sample:
        spec.n_sample = args.n_sample
    spec.key_layout = args.key_layout
    spec.parents = getattr(args, "parents", "contiguous")
    spec.elem = getattr(args, "elem", "bf16")
    return spec


def workload_text(spec, layers):
    return (f"{spec.name}: {spec.n_seqs} seq x {spec.n_q_heads} q heads / {spec.n_kv_heads} KV heads, d={spec.head_dim}, "
            f"prompt {min(spec.prompt_len)}..{max(spec.prompt_len)}, suffix cap {spec.suffix_cap}, "
            f"P={spec.parent_size}, R={spec.reps_per_parent}, K={spec.n_sample}, keys {spec.key_layout}, "
            f"{getattr(spec, 'parents', 'contiguous')} parents, {spec.elem} inputs, {layers} layers round-robin")


# -------------------------------------------------------------------------------------------
# Clock sampling (read-only NVML queries)
# -------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, device_index):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
                ids = [x for x in vis.split(",") if x.strip() != ""]
                phys = int(ids[device_index]) if ids and ids[device_index].isdigit() else device_index
                self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as e:  # NVML unavailable: report that, do not guess
            self.err = repr(e)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.ok:
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml_unavailable"]}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit and name != "gpu_idle"]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples)}


# -------------------------------------------------------------------------------------------
# The reference arm: the CPU oracle, as it stands, on the host cores
# -------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import santapp_oracle as orc
    from paper_2609_35629_b200 import synth
    spec = make_spec(args, seed=0)
    cores = len(os.sched_getaffinity(0))
    data = synth.make_layer(spec, layer=0, keep_centres=(spec.query_kind == "concentrated"))
    scale = 1.0 / math.sqrt(spec.head_dim)
    b = 0
    r0, r1 = int(data.seq_row_off[b]), int(data.seq_row_off[b + 1])
    k = synth.to_f64(data.k_prompt[:, r0:r1], spec.elem)
    v = synth.to_f64(data.v_prompt[:, r0:r1], spec.elem)
    recs = [orc.build_teams_contiguous(k[j], spec.parent_size, spec.reps_per_parent)
            for j in range(spec.n_kv_heads)]
    M = np.array([len(r[0]) - 1 for r in recs], dtype=np.int32)
    ts = np.zeros((spec.n_kv_heads, int(M.max()) + 1), dtype=np.int32)
    tm = np.zeros((spec.n_kv_heads, r1 - r0), dtype=np.int32)
    rk = np.zeros((spec.n_kv_heads, int(M.max()), spec.head_dim))
    for j, (s, m, rep) in enumerate(recs):
        ts[j, :len(s)] = s
        tm[j] = m
        rk[j, :len(rep)] = k[j][rep]

    def one(step):
        q = synth.to_f64(synth.make_queries(spec, data, step)[b], spec.elem)
        t = int(spec.suffix_len(step)[b])
        ks = synth.to_f64(data.k_suffix[b, :, :t], spec.elem) if t else None
        vs = synth.to_f64(data.v_suffix[b, :, :t], spec.elem) if t else None
        t0 = time.perf_counter()
        orc.decode_step(q, k, v, M, ts, tm, rk, ks, vs, spec.n_sample, 0, step, b, scale, n_threads=cores)
        return time.perf_counter() - t0

    for s in range(args.warmup):
        one(s)
    times = [one(args.warmup + s) for s in range(args.steps)]
    us = 1e6 * float(np.sum(times)) / max(len(times), 1)
    sample = (f"{args.steps} layer-steps of sequence 0 of layer 0 ({spec.n_q_heads} heads, {r1 - r0} prompt rows), "
              f"fp64 oracle, OpenMP over heads")
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_text(spec, 1)},
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# -------------------------------------------------------------------------------------------
# Our arm
# -------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2609_35629_b200 import binding as sp
    from paper_2609_35629_b200 import replicas

    rank, world, local_rank = replicas.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init_replicas("nccl", dev)
    sp.load_library()

    if args.workload == "latent_8k":
        res = measure_latent(args, min(args.layers, 4), min(args.steps, 20), args.warmup, dev, n_seqs=args.latent_seqs,
                             n_sample=args.n_sample or 128)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "n_gpus": world, "higher_is_better": False, "scaling": "weak",
                              "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": {"workload": res["workload"]},
                              **res}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return
    line = measure_workload(args, args.workload, args.layers, args.steps, args.warmup, dev,
                            want_e2e=not args.no_e2e, want_cpu=not args.no_cpu_baseline, want_stages=not args.no_stages)
    # Beside the headline workload (batch 1, latency-bound on this GPU), the same measurement on a
    # batch large enough to be bandwidth-bound: the ragged serving batch, two layers.
    if args.workload == "qwen7b_b1_32k" and not args.no_batched and not args.n_sample and args.key_layout == "iid":
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        big = measure_workload(args, "ragged", 2, 30, 3, dev, want_e2e=False, want_cpu=False, want_stages=True)
        if rank == 0:
            keep = ("value", "unit", "dense_us_per_layer_step", "speedup_vs_dense", "read_reduction",
                    "achieved_frac_of_peak", "dense_achieved_frac_of_peak", "roofline", "stage_us", "paired_rounds",
                    "steps", "warmup")
            line["batched"] = {"workload": big["config"]["workload"], **{k: big[k] for k in keep}}
        # the two mid-size workloads: eight 32K sequences with 64 sampled teams, and four 128K
        # sequences with 32 (a few layers and steps each)
        for key, wl, n_lay, k_over in (("mid_batch", "qwen7b_b8_32k", 4, 0), ("long_context", "long_128k", 2, 32)):
            gc.collect()
            torch.cuda.empty_cache()
            wl_args = argparse.Namespace(**{**vars(args), "n_sample": k_over})
            res = measure_workload(wl_args, wl, n_lay, 30, 3, dev, want_e2e=False, want_cpu=False, want_stages=True)
            if rank == 0:
                line[key] = {"workload": res["config"]["workload"], **{k: res[k] for k in keep}}
        # shared-latent rows (one 576-value row per token, 16 heads) at the paper's 8K study point, 32 sequences
        gc.collect()
        torch.cuda.empty_cache()
        # (budgets of the paper's study: S = 512 rows per head is K = 128 teams, S = 128 is K = 32)
        for key, k_lat in (("shared_latent", 128), ("shared_latent_k32", 32)):
            gc.collect()
            torch.cuda.empty_cache()
            lat = measure_latent(args, 2, 30, 3, dev, n_sample=k_lat)
            if rank == 0:
                line[key] = lat
        # and the headline workload with the parents of the paper's headline runs: Algorithm 3
        # (minibatch k-means with the paper's settings, fitted by the library), four layers
        if args.parents == "contiguous" and args.elem == "bf16":
            gc.collect()
            torch.cuda.empty_cache()
            km_args = argparse.Namespace(**{**vars(args), "parents": "kmeans"})
            km = measure_workload(km_args, args.workload, 4, 40, 5, dev, want_e2e=False, want_cpu=False, want_stages=True)
            if rank == 0:
                keep = ("value", "unit", "dense_us_per_layer_step", "speedup_vs_dense", "read_reduction",
                        "logical_access_pct", "roofline", "stage_us", "paired_rounds", "team_build_ms_last_layer",
                        "steps", "warmup")
                line["kmeans_parents"] = {"workload": km["config"]["workload"], **{k: km[k] for k in keep}}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def measure_workload(args, workload, n_layers, n_steps, n_warmup, dev, want_e2e, want_cpu, want_stages):
    """One workload end to end: inputs, team build, graphs, timed runs. Returns the JSON line as a
    dict on rank 0 (None elsewhere)."""
    import torch
    from paper_2609_35629_b200 import binding as sp
    from paper_2609_35629_b200 import replicas, synth

    rank, world, local_rank = replicas.env_rank_world()
    wl_args = argparse.Namespace(**{**vars(args), "workload": workload})
    # Independent replicas: every rank owns its own sequences (seed = rank); no exchange.
    spec = make_spec(wl_args, seed=replicas.replica_seed(0, rank))
    L = n_layers
    geom = sp.Geometry(spec.n_seqs, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.parent_size,
                       spec.reps_per_parent, sp.SANTAPP_FP16 if spec.elem == "fp16" else sp.SANTAPP_BF16)
    edt = geom.torch_dtype
    K = spec.n_sample
    B, Hq, Hkv, d = spec.n_seqs, spec.n_q_heads, spec.n_kv_heads, spec.head_dim
    conc = spec.query_kind == "concentrated"

    # ---- inputs: generated on the host (seeded), moved to HBM, teams built on the GPU ----
    t_prep = time.perf_counter()
    layers, host_layers = [], []
    q_all = np.empty((N_STEP_INPUTS, L, B, Hq, d), dtype=np.uint16)
    cap = max(spec.suffix_cap, 1)
    ksuf_all = torch.empty((L, B, Hkv, cap, d), dtype=edt, device=dev)
    vsuf_all = torch.empty_like(ksuf_all)
    for l in range(L):
        by_centres = spec.parents in ("centres", "kmeans")
        data = synth.make_layer(spec, layer=l, keep_centres=conc or by_centres)
        for s in range(N_STEP_INPUTS):
            q_all[s, l] = synth.make_queries(spec, data, s)
        k_prompt = sp.bf16_bits_to_cuda(data.k_prompt, dev, edt)
        v_prompt = sp.bf16_bits_to_cuda(data.v_prompt, dev, edt)
        def build_records():
            if not by_centres:
                return sp.santapp_build_teams(geom, spec.prompt_len, k_prompt, v_prompt)
            # Algorithm 3: as many centres as its first line asks for; "kmeans" fits them with the paper's
            # settings, "centres" takes the fit's ideal outcome on these keys (the centres the rows
            # were drawn around)
            n_cen = [sp.santapp_kmeans_parent_count(n, spec.parent_size) for n in spec.prompt_len]
            if spec.parents == "kmeans":
                cen_dev, _ = sp.santapp_kmeans_fit(geom, spec.prompt_len, n_cen, k_prompt)
            else:
                n_cen = [min(n, spec.n_clusters) for n in n_cen]
                cen = np.concatenate([data.centres[:, :n] for n in n_cen], axis=1)
                cen_dev = torch.from_numpy(np.ascontiguousarray(cen)).to(dev)
            parent_of = sp.santapp_assign_parents(geom, spec.prompt_len, n_cen, k_prompt, cen_dev)
            return sp.santapp_build_teams_parents(geom, spec.prompt_len, n_cen, k_prompt, v_prompt, parent_of)

        if l == L - 1:
            # the timed build is a second one, whose buffers come out of torch's cache: a first
            # build's wall clock is mostly that of fresh device allocations, which vary from run to run
            teams = build_records()
            torch.cuda.synchronize()
            del teams
        torch.cuda.synchronize()                            # the copies above are not part of the build
        t_build = time.perf_counter()
        teams = build_records()
        torch.cuda.synchronize()
        build_ms = 1e3 * (time.perf_counter() - t_build)
        del k_prompt, v_prompt
        ksuf_all[l].copy_(sp.bf16_bits_to_cuda(data.k_suffix, dev, edt))
        vsuf_all[l].copy_(sp.bf16_bits_to_cuda(data.v_suffix, dev, edt))
        layers.append(dict(teams=teams, k_suffix=ksuf_all[l], v_suffix=vsuf_all[l]))
        if l == 0:
            host_layers.append(data)
    prep_s = time.perf_counter() - t_prep

    # step s of the cycle uses decode step index (and suffix length) spread over the 256-step run
    step_ids = [int(round(i * (spec.n_steps - 1) / max(N_STEP_INPUTS - 1, 1))) for i in range(N_STEP_INPUTS)]
    sl_all = np.stack([spec.suffix_len(st) for st in step_ids]).astype(np.int32)        # [S, B]

    # packed per-step inputs: [q bytes | suffix_len | step]
    q_bytes = L * B * Hq * d * 2
    in_bytes = q_bytes + 4 * B + 4
    in_bytes_pad = (in_bytes + 255) // 256 * 256
    inputs_host = torch.zeros((N_STEP_INPUTS, in_bytes_pad), dtype=torch.uint8).pin_memory()
    for s in range(N_STEP_INPUTS):
        row = inputs_host[s].numpy()
        row[:q_bytes] = q_all[s].reshape(-1).view(np.uint8)
        row[q_bytes:q_bytes + 4 * B] = sl_all[s].view(np.uint8)
        row[q_bytes + 4 * B:in_bytes] = np.array([step_ids[s]], dtype=np.uint32).view(np.uint8)
    inputs_dev = inputs_host.to(dev)
    cur = torch.zeros(in_bytes_pad, dtype=torch.uint8, device=dev)
    q_cur = cur[:q_bytes].view(edt).view(L, B, Hq, d)
    sl_cur = cur[q_bytes:q_bytes + 4 * B].view(torch.int32)
    step_cur = cur[q_bytes + 4 * B:in_bytes].view(torch.int32)
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device=dev)
    out_dense = torch.zeros_like(out)
    ws = [torch.empty(sp.santapp_decode_workspace_bytes(geom, layers[l]["teams"], K), dtype=torch.uint8, device=dev)
          for l in range(L)]
    wsd = torch.empty(sp.santapp_dense_workspace_bytes(geom, layers[0]["teams"]), dtype=torch.uint8, device=dev)
    seed = replicas.replica_seed(1234, rank)

    def sparse_layer(l, debug=None):
        ly = layers[l]
        sp.santapp_decode_attn(geom, ly["teams"], q_cur[l], ly["k_suffix"], ly["v_suffix"], sl_cur, K, seed, 0,
                               stream_base=l * B, out=out[l], debug=debug, workspace=ws[l], step_dev=step_cur)

    def dense_layer(l):
        ly = layers[l]
        sp.santapp_dense_decode_attn(geom, ly["teams"], q_cur[l], ly["k_suffix"], ly["v_suffix"], sl_cur,
                                     out=out_dense[l], workspace=wsd)

    def set_inputs(s):
        cur.copy_(inputs_dev[s], non_blocking=True)

    # ---- accounting pass (eager): union rows per (input, layer) -> algorithmic bytes ----
    dbg = sp.DebugBuffers(geom, K, dev)
    union = np.zeros((N_STEP_INPUTS, L), dtype=np.int64)
    M_total = int(layers[0]["teams"].sizes.teams_total)                  # team slots per KV head (all are read)
    teams_real = int(layers[0]["teams"].team_count.sum().item())         # teams over all KV heads
    N_total = int(layers[0]["teams"].sizes.rows_total)
    for s in range(N_STEP_INPUTS):
        set_inputs(s)
        for l in range(L):
            sparse_layer(l, debug=dbg)
            torch.cuda.synchronize()
            union[s, l] = int(dbg.union_rows.sum().item())
            assert int(dbg.status.item()) == 0, "non-finite output"
    launches_per_layer_step = sp.santapp_last_launch_count()
    suffix_rows = sl_all.sum(axis=1).astype(np.int64) * Hkv                              # per input, per layer
    row_bytes = 2 * d * 2                                                                # K row + V row, bf16
    io_bytes = B * Hq * d * (2 + 4)                                                      # q in, out fp32
    attend_bytes = row_bytes * (union + suffix_rows[:, None]) + io_bytes                 # [S, L]
    route_bytes = Hkv * (M_total * d * 2 + (M_total + B) * 4)
    sparse_bytes = attend_bytes + route_bytes
    dense_bytes = row_bytes * (Hkv * N_total + suffix_rows) + io_bytes                   # [S]

    # ---- graphs: one decode step = all layers ----
    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for l in range(L):
                fn(l)
        return g

    set_inputs(0)
    for l in range(L):
        dense_layer(l)
    torch.cuda.synchronize()
    g_sparse = capture(sparse_layer)
    g_dense = capture(dense_layer)

    def barrier():
        replicas.barrier(dev)

    def timed(run_step, steps, warmup, sampler=None):
        for i in range(warmup):
            run_step(i)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if sampler:
            sampler.start()
        e0.record()
        for i in range(steps):
            run_step(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        if sampler:
            sampler.stop()
        ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
        barrier()
        return ms

    def sparse_step(i):
        set_inputs(i % N_STEP_INPUTS)
        g_sparse.replay()

    def dense_step(i):
        set_inputs(i % N_STEP_INPUTS)
        g_dense.replay()

    Kst, W = n_steps, max(n_warmup, 3)
    sampler = ClockSampler(local_rank)
    ms_sparse = timed(sparse_step, Kst, W, sampler)
    clocks = sampler.summary()
    n_dense = max(min(Kst, 50), 3)
    ms_dense = timed(dense_step, n_dense, 3)
    us_layer = replicas.us_per_layer_step(ms_sparse, Kst, L, world)
    us_layer_dense = replicas.us_per_layer_step(ms_dense, n_dense, L, world)

    used = np.array([(W + i) % N_STEP_INPUTS for i in range(Kst)])
    mean_sparse_bytes = float(sparse_bytes[used].mean())
    mean_attend_bytes = float(attend_bytes[used].mean())
    used_d = np.array([(3 + i) % N_STEP_INPUTS for i in range(n_dense)])
    mean_dense_bytes = float(dense_bytes[used_d].mean())

    # eager (no graph) timing of the same step, for reference
    def eager_step(i):
        set_inputs(i % N_STEP_INPUTS)
        for l in range(L):
            sparse_layer(l)
    ms_eager = timed(eager_step, max(Kst // 10, 3), 3)
    us_layer_eager = replicas.us_per_layer_step(ms_eager, max(Kst // 10, 3), L, world)

    # ---- paired rounds: sparse and dense interleaved with alternating start, median of the rounds
    # (the headline `value` above is the mean of one long region, as the output contract asks) ----
    rounds = None
    if want_stages:
        n_rounds, per_round = 6, max(min(Kst // 5, 40), 3)
        r_sparse, r_dense = [], []
        for r in range(n_rounds):
            order = (("s", sparse_step), ("d", dense_step)) if r % 2 == 0 else (("d", dense_step), ("s", sparse_step))
            for tag, fn in order:
                us = replicas.us_per_layer_step(timed(fn, per_round, 3), per_round, L, world)
                (r_sparse if tag == "s" else r_dense).append(us)
        rounds = {"n_rounds": n_rounds, "steps_per_round": per_round,
                  "sparse_us_median": float(np.median(r_sparse)), "dense_us_median": float(np.median(r_dense)),
                  "speedup_median": float(np.median(np.array(r_dense) / np.array(r_sparse))),
                  "sparse_us_min_max": [float(min(r_sparse)), float(max(r_sparse))],
                  "dense_us_min_max": [float(min(r_dense)), float(max(r_dense))]}

    # ---- isolated stages (graphs of one stage over all layers; plans and scores left in the
    # per-layer workspaces by a full step with the same inputs) ----
    stages = {}
    if want_stages:
        set_inputs(1)
        g_sparse.replay()
        torch.cuda.synchronize()
        for name, mask in (("route_score", sp.STAGE_ROUTE), ("select_plan", sp.STAGE_SELECT),
                           ("route_and_select", sp.STAGE_ROUTE | sp.STAGE_SELECT), ("attend", sp.STAGE_ATTEND),
                           ("merge", sp.STAGE_MERGE), ("attend_and_merge", sp.STAGE_ATTEND | sp.STAGE_MERGE)):
            sp.santapp_set_stage_mask(mask)
            g = capture(sparse_layer)
            sp.santapp_set_stage_mask(sp.STAGE_ALL)
            reps = max(Kst // 4, 10)
            ms = timed(lambda i: g.replay(), reps, 3)
            stages[name] = 1e3 * ms / (reps * L)                       # per launch on one GPU (slowest rank)
        attend_bytes_1 = float(attend_bytes[1].mean())
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured (MEASURED_PEAKS.json hbm_gbs)" if "hbm_gbs" in peaks else "fallback 6650 GB/s"
    roofline = None
    if stages:
        achieved = attend_bytes_1 / (stages["attend"] * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": "attend_kernel", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                    "frac": achieved / peak_gbs,
                    "traffic": (NCU_TRAFFIC_BYTES.get(spec.name)
                                if not args.n_sample and spec.key_layout == "iid" and spec.parents == "contiguous" else None),
                    "peak_kind": peak_kind,
                    "traffic_kind": "recorded from an earlier ncu capture of this kernel and workload, not measured in this run",
                    "algorithmic_bytes_per_launch": attend_bytes_1, "us_per_launch": stages["attend"],
                    "launches_timed": "attend_kernel alone (the merge kernel that follows it is stage_us.merge)"}

    # ---- end to end through host buffers ----
    e2e = None
    if want_e2e:
        new_rows = torch.zeros((N_STEP_INPUTS, 2, B, L, Hkv, d), dtype=edt).pin_memory()
        for s in range(N_STEP_INPUTS):
            for b in range(B):
                t = max(int(sl_all[s, b]) - 1, 0)
                new_rows[s, 0, b] = ksuf_all[:, b, :, t].cpu()
                new_rows[s, 1, b] = vsuf_all[:, b, :, t].cpu()
        new_dev = torch.zeros((2, B, L, Hkv, d), dtype=edt, device=dev)
        out_host = torch.zeros((L, B, Hq, d), dtype=torch.float32).pin_memory()

        def e2e_step(i):
            s = i % N_STEP_INPUTS
            cur.copy_(inputs_host[s], non_blocking=True)             # queries, suffix lengths, step
            new_dev.copy_(new_rows[s], non_blocking=True)            # the token's own K/V rows
            for b in range(B):                                       # append them to every layer's suffix
                t = max(int(sl_all[s, b]) - 1, 0)
                ksuf_all[:, b, :, t].copy_(new_dev[0, b], non_blocking=True)
                vsuf_all[:, b, :, t].copy_(new_dev[1, b], non_blocking=True)
            g_sparse.replay()
            out_host.copy_(out, non_blocking=True)
            torch.cuda.current_stream().synchronize()                # the caller reads the result

        n_e2e = max(Kst // 4, 5)
        ms_e2e = timed(e2e_step, n_e2e, 3)
        e2e = {"value": replicas.us_per_layer_step(ms_e2e, n_e2e, L, world), "unit": UNIT,
               "h2d_bytes_per_step": int(in_bytes + new_rows[0].numel() * 2),
               "d2h_bytes_per_step": int(out_host.numel() * 4)}

    # ---- the oracle on the host cores, bounded sample ----
    cpu_baseline = None
    if rank == 0 and world == 1 and want_cpu:
        cpu_baseline = cpu_baseline_leg(spec, host_layers[0], layers[0]["teams"], seed,
                                        kmeans_group_records(spec, host_layers[0], dev))

    if rank == 0:
        line = {
            "metric": METRIC, "value": us_layer, "unit": UNIT, "n_gpus": world, "steps": Kst, "warmup": W,
            "ms_per_step": ms_sparse / Kst, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": spec.elem, "data": "synthetic",
            "config": {"workload": workload_text(spec, L), "l2": "inputs larger than L2: layers visited round-robin",
                       "replay": "CUDA graph of one decode step over all layers", "replicas": world},
            "clocks": clocks, "gpu_launches": int(Kst * L * launches_per_layer_step),
            "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "layer_steps_per_s": 1e6 / us_layer, "tokens_per_s_attention_only": B * 1e6 / (us_layer * 28),
            "us_per_layer_step_eager": us_layer_eager,
            "dense_us_per_layer_step": us_layer_dense, "speedup_vs_dense": us_layer_dense / us_layer,
            "bytes_per_layer_step": mean_sparse_bytes, "dense_bytes_per_layer_step": mean_dense_bytes,
            "read_reduction": mean_dense_bytes / mean_sparse_bytes,
            "achieved_gbs": mean_sparse_bytes / (us_layer * 1e-6) / 1e9,
            "achieved_frac_of_peak": mean_sparse_bytes / (us_layer * 1e-6) / 1e9 / peak_gbs,
            "achieved_frac_of_nominal_8tbs": mean_sparse_bytes / (us_layer * 1e-6) / 8e12,
            "dense_achieved_gbs": mean_dense_bytes / (us_layer_dense * 1e-6) / 1e9,
            "dense_achieved_frac_of_peak": mean_dense_bytes / (us_layer_dense * 1e-6) / 1e9 / peak_gbs,
            "attend_bytes_per_layer_step": mean_attend_bytes,
            "logical_access_pct": 100.0 * float((teams_real + 2 * (union[used].mean() + suffix_rows[used].mean()))
                                                / (2 * (Hkv * N_total + suffix_rows[used].mean()))),
            "stage_us": stages, "paired_rounds": rounds, "prep_seconds": prep_s, "team_build_ms_last_layer": build_ms,
        }
        return line
    return None


def measure_latent(args, n_layers, n_steps, n_warmup, dev, n_seqs=32, n_sample=128):
    """Shared-latent rows (one 512 + 64 value row per token, 16 heads): the same measurement as
    measure_workload on the paper's study point (8K context, P = 16, R = 4) as a batch of sequences.
    Returns a dict on rank 0 (None elsewhere)."""
    import torch
    from paper_2609_35629_b200 import binding as sp
    from paper_2609_35629_b200 import replicas, synth

    rank, world, local_rank = replicas.env_rank_world()
    spec = synth.spec_latent_8k(seed=replicas.replica_seed(0, rank), n_seqs=n_seqs, n_sample=n_sample)
    L, B, H, K = n_layers, spec.n_seqs, spec.n_heads, spec.n_sample
    geom = sp.LatentGeometry(B, H, spec.parent_size, spec.reps_per_parent)
    ROW, DV = synth.LATENT_ROW, synth.LATENT_DIM
    scale = synth.LATENT_SCALE
    S = 4                                                   # distinct step inputs cycled through
    layers = []
    q_all = np.empty((S, L, B, H, ROW), dtype=np.uint16)
    for l in range(L):
        data = synth.make_latent_layer(spec, layer=l)
        for s in range(S):
            q_all[s, l] = synth.make_latent_queries(spec, data, s)
        rows = sp.bf16_bits_to_cuda(data.rows, dev)
        if l == L - 1:
            # the timed build is a second one, whose buffers come out of torch's cache: the first
            # build's time is mostly that of fresh device allocations (3 to 190 ms from run to run)
            teams = sp.santapp_latent_build_teams(geom, spec.prompt_len, rows)
            torch.cuda.synchronize()
            del teams
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        teams = sp.santapp_latent_build_teams(geom, spec.prompt_len, rows)
        torch.cuda.synchronize()
        build_ms = 1e3 * (time.perf_counter() - t0)
        del rows
        layers.append(dict(teams=teams, suffix=sp.bf16_bits_to_cuda(data.suffix, dev)))
    step_ids = [0, 5, 10, 15]
    sl_all = np.stack([spec.suffix_len(st) for st in step_ids]).astype(np.int32)
    q_dev = sp.bf16_bits_to_cuda(q_all, dev)
    sl_dev = torch.from_numpy(sl_all).to(dev)
    step_dev_all = torch.tensor(step_ids, dtype=torch.int32, device=dev)
    q_cur = torch.empty_like(q_dev[0])
    sl_cur = torch.empty_like(sl_dev[0])
    step_cur = torch.zeros(1, dtype=torch.int32, device=dev)
    out = torch.zeros((L, B, H, DV), dtype=torch.float32, device=dev)
    out_dense = torch.zeros_like(out)
    cap = spec.suffix_cap
    ws = [torch.empty(sp.santapp_latent_decode_workspace_bytes(geom, layers[l]["teams"], K, cap), dtype=torch.uint8, device=dev)
          for l in range(L)]
    wsd = torch.empty(sp.santapp_latent_dense_workspace_bytes(geom, layers[0]["teams"]), dtype=torch.uint8, device=dev)
    seed = replicas.replica_seed(1234, rank)

    def sparse_layer(l, debug=None):
        ly = layers[l]
        sp.santapp_latent_decode_attn(geom, ly["teams"], q_cur[l], ly["suffix"], sl_cur, K, seed, 0, scale, stream_base=l * B,
                                      out=out[l], debug=debug, workspace=ws[l], step_dev=step_cur)

    def dense_layer(l):
        ly = layers[l]
        sp.santapp_latent_dense_decode_attn(geom, ly["teams"], q_cur[l], ly["suffix"], sl_cur, scale, out=out_dense[l], workspace=wsd)

    def set_inputs(s):
        q_cur.copy_(q_dev[s], non_blocking=True)
        sl_cur.copy_(sl_dev[s], non_blocking=True)
        step_cur.copy_(step_dev_all[s:s + 1], non_blocking=True)

    dbg = sp.LatentDebugBuffers(geom, K, dev)
    union = np.zeros((S, L), dtype=np.int64)
    for s in range(S):
        set_inputs(s)
        for l in range(L):
            sparse_layer(l, debug=dbg)
            torch.cuda.synchronize()
            union[s, l] = int(dbg.union_rows.sum().item())
            assert int(dbg.status.item()) == 0, "non-finite output"
    launches = sp.santapp_last_launch_count()
    M_total = int(layers[0]["teams"].sizes.teams_total)
    N_total = int(layers[0]["teams"].sizes.rows_total)
    suffix_rows = sl_all.sum(axis=1).astype(np.int64)
    io_bytes = B * H * (ROW * 2 + DV * 4)
    attend_bytes = 2 * ROW * (union + suffix_rows[:, None]) + io_bytes              # one 1152-byte row per row read
    route_bytes = M_total * ROW * 2 + (M_total + B) * 4
    sparse_bytes = attend_bytes + route_bytes
    dense_bytes = 2 * ROW * (N_total + suffix_rows) + io_bytes

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for l in range(L):
                fn(l)
        return g

    set_inputs(0)
    for l in range(L):
        dense_layer(l)
    torch.cuda.synchronize()
    g_sparse, g_dense = capture(sparse_layer), capture(dense_layer)

    def timed(run_step, steps, warmup):
        for i in range(warmup):
            run_step(i)
        replicas.barrier(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            run_step(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
        replicas.barrier(dev)
        return ms

    def sparse_step(i):
        set_inputs(i % S)
        g_sparse.replay()

    def dense_step(i):
        set_inputs(i % S)
        g_dense.replay()

    W = max(n_warmup, 3)
    us_sparse = replicas.us_per_layer_step(timed(sparse_step, n_steps, W), n_steps, L, world)
    us_dense = replicas.us_per_layer_step(timed(dense_step, n_steps, W), n_steps, L, world)
    used = np.array([(W + i) % S for i in range(n_steps)])
    mean_sparse, mean_dense = float(sparse_bytes[used].mean()), float(dense_bytes[used].mean())
    stages = {}
    set_inputs(1)
    g_sparse.replay()
    torch.cuda.synchronize()
    for name, mask in (("route_score", sp.STAGE_ROUTE), ("select_plan", sp.STAGE_SELECT), ("attend", sp.STAGE_ATTEND),
                       ("merge", sp.STAGE_MERGE)):
        sp.santapp_set_stage_mask(mask)
        g = capture(sparse_layer)
        sp.santapp_set_stage_mask(sp.STAGE_ALL)
        reps = max(n_steps, 10)
        stages[name] = 1e3 * timed(lambda i: g.replay(), reps, 3) / (reps * L)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    attend_1 = float(attend_bytes[1].mean())
    achieved = attend_1 / (stages["attend"] * 1e-6) / 1e9
    if rank != 0:
        return None
    return {
        "workload": (f"{spec.name}: {B} seq x {H} heads sharing one {ROW}-value row per token, prompt {spec.prompt_len[0]}, "
                     f"suffix cap {cap}, P={spec.parent_size}, R={spec.reps_per_parent}, K={K}, contiguous parents, bf16, "
                     f"{L} layers round-robin"),
        "value": us_sparse, "unit": UNIT, "steps": n_steps, "warmup": W, "gpu_launches_per_layer_step": launches,
        "dense_us_per_layer_step": us_dense, "speedup_vs_dense": us_dense / us_sparse,
        "read_reduction": mean_dense / mean_sparse,
        "achieved_frac_of_peak": mean_sparse / (us_sparse * 1e-6) / 1e9 / peak_gbs,
        "dense_achieved_frac_of_peak": mean_dense / (us_dense * 1e-6) / 1e9 / peak_gbs,
        "logical_access_pct": 100.0 * float((M_total + union[used].mean() + suffix_rows[used].mean())
                                            / (N_total + suffix_rows[used].mean())),
        "roofline": {"bound": "hbm", "kernel": "latent_attend_kernel", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                     "frac": achieved / peak_gbs, "traffic": NCU_TRAFFIC_BYTES.get(spec.name) if (n_seqs, n_sample) == (32, 128) else None,
                     "algorithmic_bytes_per_launch": attend_1, "us_per_launch": stages["attend"]},
        "stage_us": stages, "team_build_ms_last_layer": build_ms,
    }


def kmeans_group_records(spec, data, dev):
    """Records of the paper's centroid-guided baseline for sequence 0: k-means groups of nominal size
    4 and 16 (Algorithm 3's fit and assignment with the paper's settings, one group per cluster routed
    by its mean key), built by the library on the GPU. Only for prompts where the greedy start of a
    fit with N / 4 centres stays within seconds."""
    import torch
    from paper_2609_35629_b200 import binding as sp
    N = int(spec.prompt_len[0])
    if N > 40000 or N < 64:
        return {}
    half = spec.elem == "fp16"
    k = sp.bf16_bits_to_cuda(np.ascontiguousarray(data.k_prompt[:, :N]), dev,
                             torch.float16 if half else torch.bfloat16)
    out = {}
    for size in (4, 16):
        geom = sp.Geometry(1, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, size, 1,
                           sp.SANTAPP_FP16 if half else sp.SANTAPP_BF16)
        n_cen = [sp.santapp_kmeans_parent_count(N, size)]
        if 3 * max(4096, n_cen[0]) > 28544:                        # the fit's limit on its initialisation sample
            continue
        centres, _ = sp.santapp_kmeans_fit(geom, [N], n_cen, k)
        labels = sp.santapp_assign_parents(geom, [N], n_cen, k, centres)
        t = sp.santapp_build_groups_mean_parents(geom, [N], n_cen, k, k, labels)
        torch.cuda.synchronize()
        cnt = t.team_count.cpu().numpy()[:, 0]
        trs, tok = t.team_row_start.cpu().numpy(), t.row_token.cpu().numpy()
        rep = t.rep_keys.view(torch.int16).cpu().numpy().view(np.uint16)
        out[f"centroid_kmeans_groups_of_{size}"] = [
            (np.ascontiguousarray(trs[j, :cnt[j] + 1]), np.ascontiguousarray(tok[j]), rep[j, :cnt[j]])
            for j in range(spec.n_kv_heads)]
    return out


def cpu_baseline_leg(spec, data, teams, seed, group_records=None):
    """The fp64 oracle on sequence 0 of layer 0, using the GPU-built team records, timed on
    all host cores for a bounded number of layer-steps."""
    from oracle import santapp_oracle as orc
    from paper_2609_35629_b200 import synth
    cores = len(os.sched_getaffinity(0))
    b = 0
    r0, r1 = int(data.seq_row_off[b]), int(data.seq_row_off[b + 1])
    n_kv, d = spec.n_kv_heads, spec.head_dim
    trs = teams.team_row_start.cpu().numpy()
    tok = teams.row_token.cpu().numpy()
    import torch
    rep_bits = teams.rep_keys.view(torch.int16).cpu().numpy().view(np.uint16)
    to = teams.seq_team_off.cpu().numpy()
    t0, t1 = int(to[b]), int(to[b + 1])
    M = np.ascontiguousarray(teams.team_count.cpu().numpy()[:, b], dtype=np.int32)     # teams of each KV head
    ts = np.ascontiguousarray(trs[:, t0 + b:t1 + b + 1])
    tm = np.ascontiguousarray(tok[:, r0:r1])
    rk = synth.to_f64(rep_bits[:, t0:t1], spec.elem)
    k = synth.to_f64(data.k_prompt[:, r0:r1], spec.elem)
    v = synth.to_f64(data.v_prompt[:, r0:r1], spec.elem)
    scale = 1.0 / math.sqrt(d)
    times, n = [], 0
    budget = time.perf_counter() + 12.0
    while time.perf_counter() < budget and n < 4000:
        step = n % spec.n_steps
        q = synth.to_f64(synth.make_queries(spec, data, step % N_STEP_INPUTS)[b], spec.elem)
        t = int(spec.suffix_len(step)[b])
        ks = synth.to_f64(data.k_suffix[b, :, :t], spec.elem) if t else None
        vs = synth.to_f64(data.v_suffix[b, :, :t], spec.elem) if t else None
        s0 = time.perf_counter()
        orc.decode_step(q, k, v, M, ts, tm, rk, ks, vs, spec.n_sample, seed, step, b, scale, n_threads=cores)
        times.append(time.perf_counter() - s0)
        n += 1
    us = 1e6 * float(np.mean(times[1:] if len(times) > 1 else times))

    # beside it, a few layer-steps each of: the oracle on one thread, and the oracle's dense
    # attention (all prompt rows) on all cores and on one thread
    def few(fn, reps):
        took = []
        for i in range(reps):
            s0 = time.perf_counter()
            fn(i)
            took.append(time.perf_counter() - s0)
        return 1e6 * float(np.mean(took))

    def inputs(i):
        step = i % spec.n_steps
        q = synth.to_f64(synth.make_queries(spec, data, step % N_STEP_INPUTS)[b], spec.elem)
        t = int(spec.suffix_len(step)[b])
        ks = synth.to_f64(data.k_suffix[b, :, :t], spec.elem) if t else None
        vs = synth.to_f64(data.v_suffix[b, :, :t], spec.elem) if t else None
        return q, ks, vs, step

    def sparse_1(i):
        q, ks, vs, step = inputs(i)
        orc.decode_step(q, k, v, M, ts, tm, rk, ks, vs, spec.n_sample, seed, step, b, scale, n_threads=1)

    def dense_n(threads):
        def run(i):
            q, ks, vs, _ = inputs(i)
            orc.dense_step(q, k, v, ks, vs, scale, n_threads=threads)
        return run

    extra = {"sparse_1_thread_us": few(sparse_1, 3), "dense_all_cores_us": few(dense_n(cores), 5),
             "dense_1_thread_us": few(dense_n(1), 2)}
    # routing agreement with dense attention over the prompt (Eq. diagnostic-kl), no sampling involved:
    # mean over the heads of two of the step inputs, for the workload's teams and for the
    # centroid-guided baseline (groups of 4 and of 16 keys routed by their mean key: contiguous
    # groups, and the k-means groups the paper's baseline uses)
    variants = {"teams": [(ts[j][:M[j] + 1], tm[j], rk[j][:M[j]]) for j in range(n_kv)]}
    for size in (4, 16):
        variants[f"centroid_groups_of_{size}"] = [orc.group_mean_keys(k[j], size, elem=spec.elem) for j in range(n_kv)]
    for name, recs in (group_records or {}).items():              # k-means groups, built by the library
        variants[name] = [(r[0], r[1], synth.to_f64(r[2], spec.elem)) for r in recs]
    kls = {name: [] for name in variants}
    for i in range(2):
        q, _, _, _ = inputs(i * 100)
        for h in range(spec.n_q_heads):
            j = h // spec.group
            for name, recs in variants.items():
                kls[name].append(orc.routing_kl(q[h], k[j], recs[j][0], recs[j][1], recs[j][2], scale))
    extra["routing_kl_nats_mean"] = {name: float(np.mean(v)) for name, v in kls.items()}
    return {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} layer-steps of sequence 0, layer 0 ({spec.n_q_heads} heads, {r1 - r0} prompt rows), "
                      f"fp64 oracle with OpenMP over heads", **extra}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
