#!/usr/bin/env python
"""Benchmark of the SSD decode path on synthetic, seeded workloads.

    python bench.py --gpus N --steps K --warmup W [--workload llada8b] [--max-drafts D]
    python bench.py --impl reference ...        # the CPU oracle, timed on the host cores

One "step" is one pass of the whole hot path over one batch: the generation of all `gen_len`
tokens of every sequence after its prompt has been prefilled (candidate selection, tree build, one
batched verification forward per iteration, acceptance, draft update, block commit, for every
block).  `value` = decode tokens/s with everything resident on the device (prefill excluded);
`e2e` = tokens/s through the host-buffer C-ABI calls, prefill and host<->device copies included.
With N > 1 every rank decodes its own replica (independent sequences, no data-path collective):
weak scaling.  Prints exactly one JSON line on rank 0.
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

METRIC = "decode tokens/s at batch 1 (LLaDA-8B-shaped) and % HBM roofline per verify forward"
# DRAM bytes per projection launch from the ncu capture summarised in
# profiles/gemm_tc_kernel_and_attn_verify_tc_llada8b_4layers_counters.md (mean over the four projections of a
# LLaDA-8B-shaped layer).
# Valid only for the kernel source it was taken from: reported as null once gemm.cu has changed.
GEMM_TRAFFIC = {"workload": "llada8b", "bytes_per_launch": 113.1e6, "gemm_cu_sha256_16": "a35294ed124f87be"}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def gemm_traffic(workload_name):
    import hashlib
    src = os.path.join(ROOT, "paper_2510_04147_b200", "csrc", "gemm.cu")
    try:
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    if sha != GEMM_TRAFFIC["gemm_cu_sha256_16"] or workload_name != GEMM_TRAFFIC["workload"]:
        return None
    return GEMM_TRAFFIC["bytes_per_launch"]


def forward_bytes(w, n_seq, S):
    """Algorithmic HBM bytes of one verification forward: every layer weight, the LM head and the
    cached prefix K/V of each sequence, each read once."""
    q, kv = w.n_heads * w.head_dim, w.n_kv_heads * w.head_dim
    per_layer = (q + 2 * kv) * w.d_model + w.d_model * q + 3 * w.d_ffn * w.d_model
    weights = 2.0 * (per_layer * w.n_layers + w.vocab * w.d_model)
    kvb = 2.0 * 2.0 * kv * w.n_layers * S * n_seq
    return weights, kvb


class ClockSampler:
    """nvidia-smi sampled during the timed region (read-only)."""

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = f"/tmp/ssd_bench_clocks_{os.getpid()}.csv"

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


# --------------------------------------------------------------------------------------------
# the CPU oracle as baseline / reference arm
# --------------------------------------------------------------------------------------------
def _oracle_threads():
    try:
        import threadpoolctl
        return max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


_HEAD_WEIGHTS = {}      # the LM-head tensors of a workload, drawn once per process (4 GB in fp64 at the 8B shapes)


def oracle_forward_times(w, layers, prefix_len, node_counts, device="cpu", with_head=True):
    """Times the oracle (as it stands) on verification forwards of `w`: for every layer index in `layers`
    the layer's tensors are drawn (outside the clock, one layer in memory at a time) and ``Oracle.layer`` is
    timed once per entry of `node_counts` (that many nodes of block_len rows against `prefix_len` cached
    positions); then the LM head on the same rows.  The inputs of a layer are seeded stand-ins (the cost of
    the oracle's arithmetic does not depend on the values).  Returns ({nodes: seconds over `layers`},
    {nodes: seconds of the LM head}, threads)."""
    import numpy as np
    import torch
    from oracle import ssd_oracle as so
    from paper_2510_04147_b200 import workloads as wl

    cfg = so.ModelConfig(w.n_layers, w.d_model, w.n_heads, w.n_kv_heads, w.head_dim, w.d_ffn, w.vocab, w.mask_id,
                         w.rope_theta, w.rms_eps)

    def draw(names):
        return {n: wl.make_tensor(w, n, device).to(torch.float32).cpu().numpy().astype(np.float64) for n in names}

    rng = np.random.default_rng(0)
    B = w.block_len
    pk = rng.standard_normal((prefix_len, w.n_kv_heads, w.head_dim))
    pv = rng.standard_normal((prefix_len, w.n_kv_heads, w.head_dim))
    t_layers = {n: 0.0 for n in node_counts}
    t_head = {n: 0.0 for n in node_counts}
    for l in layers:
        o = so.Oracle(cfg, draw([f"layers.{l}.{t}" for t in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                             "norm_attn", "norm_ffn")]))
        for n in node_counts:
            groups = [rng.standard_normal((B, w.d_model)) for _ in range(n)]
            pos = [np.arange(prefix_len, prefix_len + B) for _ in range(n)]
            t0 = time.perf_counter()
            o.layer(l, groups, pos, pk, pv)
            t_layers[n] += time.perf_counter() - t0
        del o
    if with_head:
        if w.name not in _HEAD_WEIGHTS:
            _HEAD_WEIGHTS.clear()
            _HEAD_WEIGHTS[w.name] = draw(["norm_final", "lm_head"])
        o = so.Oracle(cfg, _HEAD_WEIGHTS[w.name])
        for n in node_counts:
            h = rng.standard_normal((n * B, w.d_model))
            t0 = time.perf_counter()
            logits = so.rmsnorm(h, o._W("norm_final"), cfg.rms_eps) @ o._W("lm_head").T
            so.token_and_confidence(logits, cfg.mask_id)
            t_head[n] = time.perf_counter() - t0
            del logits
    return t_layers, t_head, _oracle_threads()


def pick_workload(args):
    """The named workload; --layers / --gen-len / --prompt-len shrink it for profiler captures only
    (such a run is labelled "reduced" and is not a benchmark of the named configuration)."""
    from paper_2510_04147_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    over = {}
    if args.layers:
        over["n_layers"] = args.layers
    if args.gen_len:
        over["gen_len"] = args.gen_len
    if args.prompt_len:
        over["prompt_len"] = args.prompt_len
    if args.batch:
        over["batch"] = args.batch
    return (w.replace(**over), True) if over else (w, False)


def run_reference(args):
    """The oracle as reference arm.  A step is a bounded sample of the workload: `--ref-layers` layers of one
    stepwise forward (one node of block_len rows against the prompt's prefix) plus the LM head, actually
    timed; step i takes the next layers in turn, so that 32 / ref-layers steps visit every layer.  `value`
    scales the mean per-layer time to the full depth (stepwise decoding: one token per forward, one commit
    forward per block); `ms_per_step` is the time the step's sample really took."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, _ = pick_workload(args)
    ls = max(1, min(args.ref_layers, w.n_layers))
    per_layer, head, step_ms = [], [], []
    device = "cpu"
    try:
        import torch
        if torch.cuda.is_available():
            device = "cuda"                     # where the seeded generator draws (its output does not depend on it)
    except Exception:
        pass
    threads = 1
    for i in range(args.warmup + args.steps):
        layers = [(i * ls + j) % w.n_layers for j in range(ls)]
        tl, th, threads = oracle_forward_times(w, layers, w.prompt_len, [1], device)
        if i >= args.warmup:
            per_layer.append(tl[1] / ls)
            head.append(th[1])
            step_ms.append(1e3 * (tl[1] + th[1]))
    t_fwd = (sum(per_layer) / len(per_layer)) * w.n_layers + sum(head) / len(head)
    tps = w.block_len / (w.block_len + 1.0) / t_fwd
    desc = (f"oracle (numpy fp64), per step {ls} of {w.n_layers} layers (next layers each step) + LM head of one stepwise "
            f"forward ({w.block_len} rows, prefix {w.prompt_len}), timed; {args.steps} steps timed; tokens/s = "
            f"block_len/(block_len+1) / (mean layer time x {w.n_layers} + LM head)")
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sum(step_ms) / len(step_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "prompt_len": w.prompt_len, "gen_len": w.gen_len, "block_len": w.block_len,
                       "batch_per_gpu": w.batch, "max_drafts": 0, "nodes_per_forward": 1,
                       "l2_policy": "inputs larger than L2 (one layer's weights are 1.7 GB in fp64)", "replicas": 1,
                       "decoding": "stepwise (oracle)", "step": f"{ls} layers + LM head of one forward",
                       "seconds_per_full_forward": t_fwd},
            "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------------
def ensure_library():
    """Compile the CUDA library when this tree has not been built yet; there is no other implementation to use."""
    from paper_2510_04147_b200 import binding, build
    if not os.path.exists(binding.LIB_PATH):
        if int(os.environ.get("LOCAL_RANK", "0")) == 0:
            build.build()
        else:                                   # another rank of this node is compiling
            t0 = time.time()
            while not os.path.exists(binding.LIB_PATH) and time.time() - t0 < 900:
                time.sleep(2.0)


def quick_workload(w, peaks, stream, drafts=(0, 1)):
    """The other configurations in short: one generation per draft length (decode tokens/s, accept
    histogram) and CUDA-event times of single forwards, on a context of its own."""
    import numpy as np
    import torch
    from paper_2510_04147_b200 import binding, workloads as wl

    B, L, P, bs = w.block_len, w.gen_len, w.prompt_len, w.batch
    ssd = binding.Ssd(binding.config_from_workload(w, max_drafts=max(drafts)))
    try:
        ssd.load_workload_weights(w, "cuda")
        ssd.prefill_dev(wl.make_prompts(w, "cuda"))
        out_tok = torch.zeros((bs, B), dtype=torch.int32).pin_memory()
        out_acc = torch.zeros((bs, B), dtype=torch.int32).pin_memory()
        out_nf = torch.zeros((bs,), dtype=torch.int32).pin_memory()
        res = {"batch": bs, "prompt_len": P, "gen_len": L, "block_len": B, "per_draft_length": {}}
        for d in drafts:
            ssd.set_option("max_drafts", d)
            mode = binding.MODE_SSD if d > 0 else binding.MODE_STEPWISE
            ssd.rewind(P)
            ssd.decode_block_into(mode, B, out_tok.data_ptr(), out_acc.data_ptr(), out_nf.data_ptr())   # warm-up block
            ssd.rewind(P)
            accs = []
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            done = 0
            while done < L:
                t = min(B, L - done)
                ssd.decode_block_into(mode, t, out_tok.data_ptr(), out_acc.data_ptr(), out_nf.data_ptr())
                accs.append(out_acc.numpy()[:, :t].copy())
                done += t
            ev1.record(stream)
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1)
            a = np.concatenate([x.reshape(-1) for x in accs])
            a = a[a > 0]
            # one forward of this chain length in the middle of a block, CUDA events around the step
            ssd.rewind(P)
            ssd.block_begin(B)
            ssd.block_step(d, bs)
            times = []
            for _ in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                acc, nn = ssd.block_step(d, bs)
                e1.record(stream)
                torch.cuda.synchronize()
                if acc.sum() == 0:
                    break
                times.append(e0.elapsed_time(e1))
            tmed = statistics.median(times)
            wb, kvb = forward_bytes(w, bs, P)
            rows = bs * (d + 1) * B
            t_hbm = (wb + kvb) / (peaks["hbm_gbs"] * 1e9)
            t_tc = 2.0 * rows * (wb / 2.0) / (peaks["bf16_tflops_sustained"] * 1e12)
            res["per_draft_length"][str(d)] = {
                "tokens_per_s": bs * L / (ms * 1e-3), "ms_per_generation": ms, "forwards_per_sequence": int(len(a) / bs),
                "mean_accepted_per_forward": float(a.mean()), "accept_histogram": np.bincount(a).tolist(),
                "forward": {"rows": rows, "ms": tmed, "algorithmic_gb": (wb + kvb) / 1e9, "hbm_frac": t_hbm / (tmed * 1e-3),
                            "frac_of_max_hbm_tensor": max(t_hbm, t_tc) / (tmed * 1e-3)}}
        best = max(res["per_draft_length"], key=lambda k: res["per_draft_length"][k]["tokens_per_s"])
        res["best_draft_length"] = int(best)
        res["tokens_per_s"] = res["per_draft_length"][best]["tokens_per_s"]
        return res
    finally:
        ssd.destroy()


def run_ours(args):
    ensure_library()
    import numpy as np
    import torch
    from paper_2510_04147_b200 import binding, replicas, workloads as wl

    rank, world, local = replicas.rank_world_local()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    w, reduced = pick_workload(args)
    B, L, P, bs = w.block_len, w.gen_len, w.prompt_len, w.batch
    n_blocks = -(-L // B)
    sweep_drafts = sorted({(w.block_len - 2 if x == "full" else int(x)) for x in args.sweep.split(",")}) if args.sweep else []
    sweep_drafts = [d for d in sweep_drafts if 0 <= d <= w.block_len - 1 and w.batch * (d + 1) * w.block_len <= 1024]
    # the full chain of a block (N = B - 2 drafts, B - 1 nodes) is timed once per run against the tensor
    # roofline; batches whose full chain would exceed 1024 rows get the longest chain within 1024 rows
    ft_nodes = max(1, min(w.block_len - 1, 1024 // (w.batch * w.block_len)))
    cfg_drafts = max([args.max_drafts if args.max_drafts >= 0 else 0] + sweep_drafts + [3, ft_nodes - 1])
    # a stream of its own (not the legacy default stream) so that dependent launches may overlap
    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)
    ssd = binding.Ssd(binding.config_from_workload(w, max_drafts=min(cfg_drafts, B - 1)))
    for k, v in (("split_k_qkv", args.split_qkv), ("split_k_o", args.split_o), ("split_k_down", args.split_down),
                 ("kv_split", args.kv_split), ("attn_impl", args.attn_impl), ("two_sm_rows", args.two_sm_rows),
                 ("gemm_max_stages", args.gemm_max_stages), ("attn_pipe_keys", args.attn_pipe_keys),
                 ("attn_pipe_ctas", args.attn_pipe_ctas)):
        if v is not None:
            ssd.set_option(k, v)
    t0 = time.time()
    ssd.load_workload_weights(w, "cuda")
    torch.cuda.synchronize()
    t_load = time.time() - t0
    # per-rank prompts: rank r decodes sequences r*bs .. r*bs+bs-1 of the seeded prompt set
    prompts = replicas.shard_prompts(w, rank, world, bs)
    prompts_pinned = prompts.clone().pin_memory()
    prompts_dev = prompts.cuda()
    out_tok = torch.zeros((bs, B), dtype=torch.int32).pin_memory()
    out_acc = torch.zeros((bs, B), dtype=torch.int32).pin_memory()
    out_nf = torch.zeros((bs,), dtype=torch.int32).pin_memory()

    def decode_all(max_drafts, collect=None):
        """All blocks of one generation through ssd_decode_block (cache must hold exactly the prompt)."""
        ssd.set_option("max_drafts", max_drafts)
        mode = binding.MODE_SSD if max_drafts > 0 else binding.MODE_STEPWISE
        done = 0
        while done < L:
            t = min(B, L - done)
            ssd.decode_block_into(mode, t, out_tok.data_ptr(), out_acc.data_ptr(), out_nf.data_ptr())
            if collect is not None:
                collect.append(out_acc.numpy()[:, :t].copy())
            done += t

    def timed_generation(max_drafts, reps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(reps):
            ssd.rewind(P)
            decode_all(max_drafts)
        ev1.record(stream)
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / reps

    def accept_stats(max_drafts):
        hist = []
        ssd.rewind(P)
        decode_all(max_drafts, hist)
        accs = np.concatenate([a.reshape(-1) for a in hist])
        return accs[accs > 0]

    t0 = time.time()
    ssd.prefill_dev(prompts_dev)
    torch.cuda.synchronize()
    t_prefill = time.time() - t0

    # ---- choose the draft length: quick sweep (untimed for the headline), or the one given
    sweep = {}
    if args.max_drafts >= 0:
        best = args.max_drafts
    else:
        for d in sweep_drafts:
            ms = timed_generation(d, 1)
            accs = accept_stats(d)
            sweep[str(d)] = {"tokens_per_s": bs * L / (ms * 1e-3), "ms_per_generation": ms,
                             "mean_accepted_per_forward": float(accs.mean()), "forwards": int(len(accs))}
        best = int(max(sweep, key=lambda k: sweep[k]["tokens_per_s"]))
    # the configured cap decides buffer sizes only; the draft length used is `best`
    for _ in range(args.warmup):
        ssd.rewind(P)
        decode_all(best)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = ClockSampler(local)
    clocks.start()
    launches0 = ssd.launch_count()
    torch.cuda.synchronize()
    ms = timed_generation(best, args.steps)
    launches = ssd.launch_count() - launches0
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clk = clocks.stop()
    ms = replicas.max_over_ranks(ms, dist, "cuda")
    value = replicas.job_tokens_per_s(world, bs, L, ms)

    # ---- end to end: host prompt -> prefill -> all blocks with host outputs, every step
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(1, args.steps)
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(e2e_steps):
        ssd.prefill_ptr(bs, P, prompts_pinned.data_ptr())
        decode_all(best)
    ev1.record(stream)
    torch.cuda.synchronize()
    ms_e2e = ev0.elapsed_time(ev1) / e2e_steps
    ms_e2e = replicas.max_over_ranks(ms_e2e, dist, "cuda")
    e2e_value = replicas.job_tokens_per_s(world, bs, L, ms_e2e)

    line = None
    if rank == 0:
        # ---- accept statistics of the timed configuration
        accs = accept_stats(best)
        # ---- per-forward roofline: stepwise (1 node) and the chosen chain, CUDA events per forward
        fwd = {}
        labels = [("stepwise_1_node", 0), (f"ssd_{best + 1}_nodes", best)]
        for extra in (1, 3):                            # 2 and 4 nodes always: forward time against the row count
            if extra != best and extra + 1 <= ft_nodes:
                labels.append((f"ssd_{extra + 1}_nodes", extra))
        labels.append(("full_tree", ft_nodes - 1))
        for label, d in labels:
            ssd.set_option("max_drafts", d)
            ssd.rewind(P)
            ssd.block_begin(B)
            ssd.block_step(d, bs)                       # root-only forward creates the drafts
            times = []
            nodes = []
            for it in range(6):
                if label == "full_tree" and it > 0:     # only the first step after the root has the full chain
                    ssd.rewind(P)
                    ssd.block_begin(B)
                    ssd.block_step(d, bs)
                    if it >= 3:
                        break
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                acc, nn = ssd.block_step(d, bs)
                e1.record(stream)
                torch.cuda.synchronize()
                if acc.sum() == 0:
                    break
                times.append(e0.elapsed_time(e1))
                nodes.append(int(nn.max()))
            tmed = statistics.median(times)
            wb, kvb = forward_bytes(w, bs, P)
            rows = bs * max(nodes) * B
            fl = 2.0 * rows * (wb / 2.0)
            t_hbm = (wb + kvb) / (peaks["hbm_gbs"] * 1e9)
            t_tc = fl / (peaks["bf16_tflops_sustained"] * 1e12)
            fwd[label] = {"nodes": max(nodes), "rows": rows, "ms": tmed, "algorithmic_gb": (wb + kvb) / 1e9,
                          "hbm_frac": t_hbm / (tmed * 1e-3), "frac_of_max_hbm_tensor": max(t_hbm, t_tc) / (tmed * 1e-3)}
        # what a chain is worth when every draft is accepted (Table 2's upper bound: n tokens per forward of n
        # nodes): n x (one-node forward time) / (n-node forward time).  The acceptance of a random-init model
        # is far lower; this bounds what the forward's row dependence leaves of the method's speed-up.
        t1 = fwd["stepwise_1_node"]["ms"]
        for label, f in fwd.items():
            if label.startswith("ssd_"):
                f["speedup_over_stepwise_if_every_draft_accepted"] = f["nodes"] * t1 / f["ms"]
        # ---- dominant kernel: the projection GEMM family, CUDA events around every launch
        ssd.set_option("max_drafts", best)
        ssd.rewind(P)
        ssd.block_begin(B)
        ssd.block_step(best, bs)
        ssd.profile_enable(True)
        ssd.profile_read()
        for _ in range(3):
            ssd.block_step(best, bs)
        prof = ssd.profile_read()
        ssd.profile_enable(False)
        # ---- the same forwards in the live stream: every launch charged from its predecessor's end to its own
        ssd.profile_enable(2)
        for _ in range(3):
            ssd.block_step(best, bs)
        live = ssd.profile_read()
        ssd.profile_enable(False)
        lg = live["gemm"]
        live_total = sum(live[k]["ms"] for k in binding.PROF_TOP)
        in_stream = {"method": "marker kernel behind every launch; a launch is charged from the completion of its "
                               "predecessor to its own completion (adds ~1 us of dependency latency per launch)",
                     "achieved": lg["bytes"] / (lg["ms"] * 1e-3) / 1e9 if lg["ms"] > 0 else 0.0,
                     "avg_launch_us": 1e3 * lg["ms"] / max(1, lg["launches"]),
                     "family_avg_launch_us": {k: 1e3 * live[k]["ms"] / max(1, live[k]["launches"]) for k in binding.PROF_TOP},
                     "family_share_of_device_time": {k: (live[k]["ms"] / live_total if live_total else 0) for k in binding.PROF_TOP},
                     "per_projection": {k: {"avg_launch_us": 1e3 * v["ms"] / max(1, v["launches"]),
                                            "gb_per_s": (v["bytes"] / (v["ms"] * 1e-3) / 1e9 if v["ms"] > 0 else 0.0)}
                                        for k, v in live.items() if k not in binding.PROF_TOP}}
        in_stream["frac"] = in_stream["achieved"] / peaks["hbm_gbs"]
        g = prof["gemm"]
        achieved = g["bytes"] / (g["ms"] * 1e-3) / 1e9 if g["ms"] > 0 else 0.0
        total_ms = sum(prof[k]["ms"] for k in binding.PROF_TOP)
        per_projection = {k: {"launches": v["launches"], "avg_launch_us": 1e3 * v["ms"] / max(1, v["launches"]),
                              "gb_per_s": (v["bytes"] / (v["ms"] * 1e-3) / 1e9 if v["ms"] > 0 else 0.0)}
                          for k, v in prof.items() if k not in binding.PROF_TOP}
        roofline = {"bound": "hbm", "kernel": "gemm_tc_kernel (QKV/O/gate-up/down projections)",
                    "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                    "peak_source": peaks["_source"], "traffic": gemm_traffic(args.workload) if not reduced else None,
                    "launches": g["launches"], "avg_launch_us": 1e3 * g["ms"] / max(1, g["launches"]),
                    "bytes_per_launch_avg": g["bytes"] / max(1, g["launches"]),
                    "family_share_of_device_time": {k: (prof[k]["ms"] / total_ms if total_ms else 0)
                                                    for k in binding.PROF_TOP},
                    "family_avg_launch_us": {k: 1e3 * prof[k]["ms"] / max(1, prof[k]["launches"]) for k in binding.PROF_TOP},
                    "per_projection": per_projection, "in_stream": in_stream}
        # ---- the method's variants at the chosen draft length (one generation each; same tokens as stepwise
        #      decoding, under the dual cache: as stepwise decoding with the same refresh schedule)
        variants = {}

        def one_generation(d, cross_block=False):
            hist, toks = [], []
            ssd.set_option("max_drafts", d)
            mode = binding.MODE_SSD if d > 0 else binding.MODE_STEPWISE
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            done = 0
            while done < L:
                t = min(B, L - done)
                if cross_block:
                    ssd.set_option("cross_block", min(B, L - done - t))
                ssd.decode_block_into(mode, t, out_tok.data_ptr(), out_acc.data_ptr(), out_nf.data_ptr())
                hist.append(out_acc.numpy()[:, :t].copy())
                toks.append(out_tok.numpy()[:, :t].copy())
                done += t
            ev1.record(stream)
            torch.cuda.synchronize()
            a = np.concatenate([x.reshape(-1) for x in hist])
            a = a[a > 0]
            return {"tokens_per_s": bs * L / (ev0.elapsed_time(ev1) * 1e-3), "forwards": int(len(a)),
                    "mean_accepted_per_forward": float(a.mean()), "_tokens": np.concatenate(toks, axis=1)}

        def same_tokens(res, ref):
            """Share of the generation (from its start) that equals the reference decoding, token for token."""
            neq = np.nonzero(res["_tokens"].reshape(-1) != ref["_tokens"].reshape(-1))[0]
            return 1.0 if len(neq) == 0 else float(neq[0]) / res["_tokens"].size

        try:
            dv = max(best, 2)
            ssd.rewind(P)
            ref_step = one_generation(0)
            ssd.rewind(P)
            ssd.set_option("mix_order", 1)
            variants[f"mix_order_tree_{dv}_drafts"] = one_generation(dv)
            ssd.set_option("mix_order", 0)
            ssd.rewind(P)
            variants[f"greedy_chain_{dv}_drafts"] = one_generation(dv)
            ssd.rewind(P)
            variants[f"cross_block_{max(best, 1)}_drafts"] = one_generation(max(best, 1), cross_block=True)
            ssd.set_option("cross_block", 0)
            ssd.rewind(P)
            ssd.set_option("dual_cache", P + L)
            ssd.set_option("refresh_interval", 8)
            r0 = ssd.refresh_count()
            variants["dual_cache_refresh_8_stepwise"] = one_generation(0)
            variants["dual_cache_refresh_8_stepwise"]["refresh_forwards"] = ssd.refresh_count() - r0
            ssd.set_option("dual_cache", 0)
            ssd.rewind(P)
            ssd.set_option("dual_cache", P + L)
            r0 = ssd.refresh_count()
            variants[f"dual_cache_refresh_8_ssd_{max(best, 1)}_drafts"] = one_generation(max(best, 1))
            variants[f"dual_cache_refresh_8_ssd_{max(best, 1)}_drafts"]["refresh_forwards"] = ssd.refresh_count() - r0
            ssd.set_option("dual_cache", 0)
            ssd.rewind(P)
            # losslessness on the device: the share of the generation that equals stepwise decoding from its start
            # (1.0 = all of it; with candidates from the next block a decision that is a near-tie within rounding noise
            # may fall the other way at a block boundary, after which the two decodings are not comparable)
            for k, v in variants.items():
                ref = variants["dual_cache_refresh_8_stepwise"] if k.startswith("dual_cache") else ref_step
                v["leading_share_equal_to_stepwise"] = same_tokens(v, ref)
            for v in variants.values():
                v.pop("_tokens", None)
        except Exception as e:                    # a variant that does not fit this configuration is reported, not fatal
            for v in variants.values():
                if isinstance(v, dict):
                    v.pop("_tokens", None)
            variants["error"] = str(e)
            for k, v in (("mix_order", 0), ("cross_block", 0), ("dual_cache", 0)):
                try:
                    ssd.set_option(k, v)
                except Exception:
                    pass
        # ---- CPU baseline: the oracle on a bounded sample
        if args.no_cpu_baseline:
            cpu = None
        else:
            nodes_timed = sorted({1, best + 1})
            tl, th, threads = oracle_forward_times(w, range(w.n_layers), P, nodes_timed, "cuda")
            t_fwd = tl[1] + th[1]                               # one stepwise forward, every layer timed
            t_ver = tl[best + 1] + th[best + 1]                 # one verification forward of the benchmarked chain
            desc = (f"oracle (numpy fp64), {w.n_layers} of {w.n_layers} layers + LM head actually timed, once as a stepwise "
                    f"forward (1 node, {B} rows) and once as the verification forward of the benchmarked chain "
                    f"({best + 1} nodes), prefix {P}; weights drawn one layer at a time outside the clock; value = "
                    f"stepwise tokens/s = block_len/(block_len+1) / forward time (one token per forward, one commit per block)")
            cpu = {"value": B / (B + 1.0) / t_fwd, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                   "sample": desc, "seconds_per_forward": t_fwd, "seconds_per_verify_forward": t_ver,
                   "ssd_tokens_per_s_at_measured_acceptance": float(accs.mean()) / t_ver}
        line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": w.name, "prompt_len": P, "gen_len": L, "block_len": B, "batch_per_gpu": bs,
                           "max_drafts": best, "nodes_per_forward": best + 1,
                           "l2_policy": "inputs larger than L2 (15 GB of weights streamed per forward)",
                           "replicas": world, "weights_load_s": t_load, "prefill_s": t_prefill,
                           **({"reduced_for_profiling": {"n_layers": w.n_layers, "gen_len": L, "prompt_len": P}}
                              if reduced else {})},
                "clocks": clk, "gpu_launches": int(launches),
                "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": int(bs * P * 4),
                        "d2h_bytes_per_step": int(n_blocks * bs * (2 * B + 1) * 4), "ms_per_step": ms_e2e,
                        "includes": "host prompt copy + prefill + every block's tokens/accept counts read back"},
                "roofline": roofline, "forward": fwd, "cpu_baseline": cpu,
                "accept": {"mean_per_forward": float(accs.mean()), "histogram": np.bincount(accs).tolist(),
                           "forwards_per_generation": int(len(accs)), "blocks": n_blocks},
                "sweep": sweep, "variants": variants,
                "paper_context": "paper reports 2.0-3.46x over stepwise decoding on one A100 80GB with trained weights"}
    ssd.destroy()
    if line is not None and world == 1 and not reduced and args.workload == "llada8b" and not args.no_other_workloads:
        # the other configurations, each on a context of its own (one generation per draft length)
        others = {}
        torch.cuda.empty_cache()
        for name, batches in (("dream7b", (1,)), ("llada8b_batch", (1, 2, 4, 8)), ("llada8b_long", (4,))):
            for b in batches:
                wo = wl.WORKLOADS[name].replace(batch=b)
                key = name if len(batches) == 1 else f"{name}_{b}"
                try:
                    others[key] = quick_workload(wo, peaks, stream)
                except Exception as e:                    # report, do not lose the headline line
                    others[key] = {"error": str(e)}
                torch.cuda.empty_cache()
        line["workloads"] = others
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b")
    ap.add_argument("--max-drafts", type=int, default=-1, help="draft length N; -1: pick the best of --sweep")
    ap.add_argument("--sweep", default="0,1,3,5,7,full", help="draft lengths tried; full = block_len - 2 (the whole block as one chain)")
    ap.add_argument("--ref-layers", type=int, default=4, help="--impl reference: layers timed per step")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--split-qkv", type=int, default=None)
    ap.add_argument("--split-o", type=int, default=None)
    ap.add_argument("--split-down", type=int, default=None)
    ap.add_argument("--kv-split", type=int, default=None)
    ap.add_argument("--attn-impl", type=int, default=None, help="0: mma.sync attention; 1: tcgen05 attention where eligible")
    ap.add_argument("--two-sm-rows", type=int, default=None,
                    help="projection tile pairs run as one two-SM MMA from this many rows on (0: never)")
    ap.add_argument("--gemm-max-stages", type=int, default=None, help="tuning: cap on the projection kernel's ring depth")
    ap.add_argument("--attn-pipe-keys", type=int, default=None,
                    help="tuning: prefixes of at least this many keys take the pipelined attention form (0: never)")
    ap.add_argument("--attn-pipe-ctas", type=int, default=None,
                    help="tuning: ... when the batch gives it at least this many (head, sequence) CTAs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="profiling only: fewer layers of the same shape")
    ap.add_argument("--gen-len", type=int, default=0, help="profiling only: shorter generation")
    ap.add_argument("--prompt-len", type=int, default=0, help="profiling only: another prompt length")
    ap.add_argument("--batch", type=int, default=0, help="profiling only: another batch size")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
