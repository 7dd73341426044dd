#!/usr/bin/env python
"""Benchmark of the batch-1 decode step: ms/token and achieved fraction of the HBM roofline.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One "step" is one decode step (one token) of the named decoder shape over its pre-filled KV cache,
i.e. one replay of the step graph.  The default workload is the Qwen2.5-1.5B-shaped decoder with a
2048-position cache.  With N > 1 (torchrun) every rank runs an independent replica of the same
request (the step does not shard; there is no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np

from edgefm_synth import CONFIGS, GLOBAL_SEED, first_token, make_kv, make_weights

# DRAM traffic of one launch of the step kernel: dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of
# that kernel, per configuration, with the profile summary (and the source revision it names) the figure comes from.
# Only captured configurations have a value; a figure is only as current as its summary says.
NCU_TRAFFIC = {"qwen2.5-1.5b": {"bytes": None, "source": "profiles/decode_megakernel_qwen2.5-1.5b_ctx2048.md"}}


def ncu_traffic(name):
    """(bytes or None, where the figure comes from): parsed from the profile summary, which states read and write bytes."""
    import re
    ent = NCU_TRAFFIC.get(name)
    if not ent:
        return None, None
    path = ROOT / ent["source"]
    try:
        text = path.read_text()
        rd = re.search(r"dram__bytes_read\.sum\s*\|\s*([0-9.]+)\s*GB", text)
        wr = re.search(r"dram__bytes_write\.sum\s*\|\s*([0-9.]+)\s*MB", text)
        rev = re.search(r"source revision:\s*`?([0-9a-f]{7,40})", text)
        if rd and wr:
            return float(rd.group(1)) * 1e9 + float(wr.group(1)) * 1e6, f"{ent['source']}" + (f" (revision {rev.group(1)})" if rev else "")
    except OSError:
        pass
    return None, None

METRIC = "batch1_decode_ms_per_token"
UNIT = "ms/token"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json, torch copy read+write)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi sampled every 200 ms while the timed region runs (read-only queries)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.gpu)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in Path(self.path).read_text().splitlines():
                c = [x.strip() for x in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for n, val in zip(names, c[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(cfg, weights, k, v, steps: int, warmup: int, kv_format: str = "bf16"):
    """The CPU oracle as it stands, on the host cores: `steps` decode steps from the configured cache."""
    from oracle import OracleModel
    m = OracleModel(cfg, weights, cfg.cache_len + steps + warmup, kv_format=kv_format)
    m.load_kv(k, v)
    tok, pos = first_token(cfg), cfg.first_position
    for _ in range(warmup):
        _, tok = m.step(tok, pos); pos += 1
    t0 = time.perf_counter()
    for _ in range(steps):
        _, tok = m.step(tok, pos); pos += 1
    dt = time.perf_counter() - t0
    m.close()
    return dt / steps * 1e3


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    os.environ["OMP_NUM_THREADS"] = str(cores)
    weights = make_weights(cfg)
    k, v = make_kv(cfg)
    ms = time_oracle(cfg, weights, k, v, args.steps, args.warmup, args.kv_format)
    sample = f"{args.steps} full oracle decode steps of {cfg.name} from a {cfg.cache_len}-position cache (fp64 accumulation)"
    line = {"impl": "reference", "metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64 accumulate over bf16 weights", "data": "synthetic",
            "config": config_block(cfg, workload_name(cfg, args.kv_format), 1),
            "cpu_baseline": {"value": ms, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": ms, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def config_block(cfg, workload, world, pruned_bytes=0):
    """The `config` object of the JSON line (the same keys for both arms)."""
    return {"workload": workload, "replicas": world,
            "l2": (f"working set {(cfg.mean_step_bytes() - pruned_bytes) / 1e9:.2f} GB per step exceeds the 126 MB L2; no flush"
                   if cfg.mean_step_bytes() > 2.5e8 else "working set fits L2: NOT an HBM measurement"),
            "seed": GLOBAL_SEED}


def max_over_ranks(times, world):
    """Element-wise maximum over the ranks of a 1-D float64 tensor of this rank's timings (the slowest replica decides).
    N = 1: the tensor itself."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    return times


def per_token_stats(seq_ms, steps, world):
    """Median and minimum ms per token over the timed sequences (each entry: max over ranks of one sequence's time);
    with N replicas N * steps tokens leave the job per sequence."""
    per = sorted(float(t) / (steps * world) for t in seq_ms)
    return statistics.median(per), per[0]


def kv_saved_bytes(cfg, cur_len: int) -> int:
    """Bytes the compressed cache (head_dim codes + one fp32 scale per row instead of 2 head_dim bytes) saves per step at
    cache length cur_len: cur_len + 1 rows of K and of V read and one written, per layer and kv head."""
    return 2 * cfg.n_layers * cfg.n_kv_heads * (cfg.head_dim - 4) * (cur_len + 2)


def workload_name(cfg, kv_format="bf16"):
    cache = "bf16" if kv_format == "bf16" else "compressed (8-bit codes + fp32 scale per row)"
    return (f"{cfg.name}-shaped decoder, batch 1, {cfg.cache_len}-position {cache} KV cache, greedy decode steps "
            f"(L={cfg.n_layers} H={cfg.hidden} heads={cfg.n_q_heads}/{cfg.n_kv_heads} d={cfg.head_dim} F={cfg.ffn} V={cfg.vocab})")


def run_block(args, cfg):
    """Block verification (edgefm_verify_block, blocks of two): ms per GENERATED token when every call carries the token to
    decode and a proposal.  There is no draft model here: the proposals are the model's own greedy continuation, recorded in
    an untimed plain run (so they are accepted unless --reject-every spoils some, or the two kernel builds round a near-tie
    differently); the tokens generated are counted from the cache length the device reports.  One GPU."""
    import torch
    from paper_2604_27476_b200 import DecodeContext, build as cuda_build, upload_weights
    cuda_build.build()
    dev = "cuda:0"
    steps = args.steps
    weights = make_weights(cfg)
    k, v = make_kv(cfg)
    ptrs, keep = upload_weights(weights, dev)
    B = args.block_tokens
    dense = B > 4          # blocks of more than four tokens take the dense path (prefill kernels) on a plain context; every call then
                           # reads the accepted length and the next token back to the host (part of the timed loop)
    ctx = DecodeContext(cfg, ptrs, cfg.cache_len + B * steps + B + 2, dev, block_tokens=0 if dense else B)
    kd = torch.from_numpy(k.view(np.int16)).to(dev)
    vd = torch.from_numpy(v.view(np.int16)).to(dev)
    tok0, pos0 = first_token(cfg), cfg.first_position
    # the greedy continuation, by plain steps on the same context (untimed)
    ctx.prefill_kv(kd, vd)
    seq = [tok0]
    ctx.step(tok0, pos0, want_logits=False)
    for _ in range(B * steps + B):
        torch.cuda.synchronize()
        seq.append(int(ctx.next_token.item()))
        ctx.step(-1, -1, want_logits=False)
    torch.cuda.synchronize()

    def one_sequence():
        """`steps` calls; returns the tokens that entered the cache."""
        ctx.prefill_kv(kd, vd)
        idx = 0                      # seq[idx] is the token the next call decodes (if every correct proposal is accepted)
        for c in range(steps):
            spoil = args.reject_every > 0 and c % args.reject_every == args.reject_every - 1   # the LAST proposal of this call is wrong
            props = [seq[idx + t] for t in range(1, B)]
            if spoil:
                props[-1] = (props[-1] + 1) % cfg.vocab
            if dense:
                ctx.verify_block([seq[idx]] + props, pos0 + idx, want_logits=False)
                ctx.sync_length()
            else:
                ctx.verify_block([tok0 if c == 0 else -1] + props, pos0 if c == 0 else -1, want_logits=False)
            idx += B - 1 if spoil else B
        return idx

    for _ in range(max(args.warmup_sequences, 1)):
        one_sequence()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    per_tok, accepted = [], []
    for _ in range(max(args.sequences, 1)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ctx.prefill_kv(kd, vd)
        torch.cuda.synchronize()
        # (the prefill above is outside the events; one_sequence repeats it, which costs ~20 us of 100+ ms)
        e0.record()
        one_sequence()
        e1.record()
        torch.cuda.synchronize()
        n_tok = ctx.sync_length() - cfg.cache_len
        per_tok.append(e0.elapsed_time(e1) / n_tok)
        accepted.append(n_tok / steps)
    clocks = sampler.stop()
    per_tok.sort()
    ms = statistics.median(per_tok)
    line = {"metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 0, "ms_per_step": ms * statistics.median(accepted),
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 weights/KV, fp32 accumulate" + (", activations as two bf16 pieces (16 mantissa bits)" if B > 2 else ""), "data": "synthetic",
            "config": config_block(cfg, workload_name(cfg) + f", verified in blocks of {B} tokens (proposals: the model's own greedy continuation"
                                   + (f", the last one of every {args.reject_every}th call spoiled" if args.reject_every else "") + ")", 1),
            "timed_sequences": len(per_tok), "ms_per_token_min": per_tok[0], "tokens_per_call": statistics.median(accepted),
            "tokens_per_s": 1e3 / ms, "gpu_launches": steps * len(per_tok), "clocks": clocks}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_prefill(args, cfg):
    """The prefill phase (edgefm_prefill) for a prompt of --prefill tokens into an empty cache: ms per prompt (median over
    --sequences calls, each between its own CUDA events), prompt tokens/s and the contraction rate.  Not the headline
    workload.  Flops counted: 2 * tokens * (weights of the four projections of every layer) + causal attention (4 * d * n_q * sum over
    queries of the keys seen) + the output layer for the last token."""
    import torch
    from paper_2604_27476_b200 import DecodeContext, build as cuda_build, upload_weights
    cuda_build.build()
    dev = "cuda:0"
    T = args.prefill
    weights = make_weights(cfg)
    ptrs, keep = upload_weights(weights, dev)
    ctx = DecodeContext(cfg, ptrs, T + 2, dev, kv_format=None if args.kv_format == "bf16" else args.kv_format)
    toks = np.random.default_rng(1).integers(0, cfg.vocab, T).tolist()
    for _ in range(max(args.warmup_sequences, 3)):
        ctx.reset()
        ctx.prefill(toks, 0, want_logits=False)
    torch.cuda.synchronize()
    ctx.sync_status()
    sampler = ClockSampler(0)
    sampler.start()
    times = []
    for _ in range(max(args.sequences, 1)):
        ctx.reset()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.prefill(toks, 0, want_logits=False)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    ctx.sync_status()
    times.sort()
    ms = statistics.median(times)
    H, F, d, nq, nkv, L = cfg.hidden, cfg.ffn, cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads, cfg.n_layers
    n = T
    qkv = (nq + 2 * nkv) * d * H
    rest = nq * d * H + 3 * H * F
    flops = 2.0 * n * L * (qkv + rest) + L * 4.0 * d * nq * (n * (n + 1) / 2) + 2.0 * cfg.vocab * H
    peaks = {}
    try:
        peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text())
    except Exception:
        pass
    peak = float(peaks.get("bf16_tflops_sustained") or 1400.0)   # a prompt is a long step: the sustained figure
    tf = flops / (ms * 1e-3) / 1e12
    line = {"metric": "prefill_ms_per_prompt", "value": ms, "unit": "ms", "n_gpus": 1, "steps": len(times), "warmup": max(args.warmup_sequences, 3),
            "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights/KV, activations as two bf16 pieces, fp32 accumulate (tcgen05)" + (", 8-bit KV cache" if args.kv_format == "int8" else ""), "data": "synthetic",
            "config": {"workload": f"{cfg.name}: prefill of {T} prompt tokens into an empty " + ("compressed (8-bit) " if args.kv_format == "int8" else "") + f"cache (edgefm_prefill: dense contractions for all tokens, the output layer for the last one)",
                       "l2": "weights (> 2.6 GB) and activations exceed L2; nothing flushed"},
            "ms_min": times[0], "prompt_tokens_per_s": T / (ms * 1e-3),
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "traffic": None,
                         "note": "achieved counts the method's flops; the tensor cores execute twice that (two bf16 pieces per activation); peak = measured sustained cuBLAS bf16 rate" + ("" if peaks.get("bf16_tflops_sustained") else " (fallback)")},
            "gpu_launches": len(times) * ctx_prefill_launches(cfg, args.kv_format == "int8"), "clocks": clocks}
    print(json.dumps(line), flush=True)
    ctx.close()


def ctx_prefill_launches(cfg, kv_int8=False):
    """Kernels one edgefm_prefill call (8 tokens or more) enqueues: rope table + embedding/norm, 7 per layer (QKV, attention, O,
    norm, gate/up, down, norm; one more per layer compresses the new rows of an 8-bit cache), the output layer."""
    return 2 + (8 if kv_int8 else 7) * cfg.n_layers + 1


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--config", default="qwen2.5-1.5b", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU-oracle timing leg")
    ap.add_argument("--cpu-steps", type=int, default=3)
    ap.add_argument("--sequences", type=int, default=10,
                    help="timed repetitions of the --steps-long greedy sequence (each timed on its own; value = median)")
    ap.add_argument("--warmup-sequences", type=int, default=3, help="untimed sequences before the timed ones (besides --warmup steps)")
    ap.add_argument("--vocab-subset", type=int, default=0,
                    help="prune the output layer to this many evenly spaced token ids (0 = full vocabulary, the headline workload)")
    ap.add_argument("--kv-format", default="bf16", choices=["bf16", "int8"],
                    help="cache format: int8 = the compressed cache (edgefm_create_with_options); not the headline configuration")
    ap.add_argument("--block-tokens", type=int, default=1, choices=[1, 2, 4, 8],
                    help="2 / 4: generate through edgefm_verify_block, that many tokens per call (not the headline configuration)")
    ap.add_argument("--reject-every", type=int, default=0, help="with --block-tokens 2: spoil every n-th proposal (0 = none)")
    ap.add_argument("--prefill", type=int, default=0,
                    help="instead of the decode benchmark: time edgefm_prefill for a prompt of this many tokens (not the headline workload)")
    ap.add_argument("--phase-timeline", action="store_true",
                    help="instead of the benchmark: print the per-operator timeline of one step from the kernel's own device timestamps")
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    if args.phase_timeline:
        from paper_2604_27476_b200 import build as cuda_build, timeline
        cuda_build.build()
        print(timeline.format_table(timeline.summarize(timeline.collect(cfg, block_tokens=args.block_tokens if args.block_tokens > 1 else 0), cfg), cfg))
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return
    if args.block_tokens > 1:
        if rank == 0:
            run_block(args, cfg)
        return
    if args.prefill > 0:
        if rank == 0:
            run_prefill(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2604_27476_b200 import DecodeContext, build as cuda_build, edgefm_decode_step, upload_weights

    if rank == 0:
        cuda_build.build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode step has no CPU path")
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
        dist.barrier()

    steps, warmup = args.steps, max(args.warmup, 0)
    weights = make_weights(cfg)
    k, v = make_kv(cfg)
    ptrs, keep = upload_weights(weights, dev)
    span = max(steps, warmup, 1)
    ctx = DecodeContext(cfg, ptrs, cfg.cache_len + span, dev, kv_format=None if args.kv_format == "bf16" else args.kv_format)
    kd = torch.from_numpy(k.view(np.int16)).to(dev)
    vd = torch.from_numpy(v.view(np.int16)).to(dev)
    stream = torch.cuda.current_stream().cuda_stream
    tok0, pos0 = first_token(cfg), cfg.first_position
    handle = ctx.handle
    n_sub = 0
    if args.vocab_subset:
        ids = np.unique(np.linspace(0, cfg.vocab - 1, min(args.vocab_subset, cfg.vocab)).astype(np.int32))
        ctx.set_vocab_subset(ids)
        n_sub = int(ids.size)
    pruned_bytes = (cfg.vocab - n_sub) * cfg.hidden * 2 if n_sub else 0      # lm_head rows the pruned step does not read
    workload = workload_name(cfg, args.kv_format) + (f", output layer pruned to {n_sub} of {cfg.vocab} token ids" if n_sub else "")

    def free_run(n):
        """n chained greedy steps, token and position carried on the device (one graph launch per token)."""
        ctx.prefill_kv(kd, vd)
        edgefm_decode_step(handle, tok0, pos0, stream, None, None)
        for _ in range(n - 1):
            edgefm_decode_step(handle, -1, -1, stream, None, None)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing (inputs in HBM; weights 3 GB >> L2, so no flush between steps) ---------
    # --warmup untimed steps, then --warmup-sequences untimed sequences, then --sequences sequences of exactly --steps
    # steps, each bracketed by its own pair of CUDA events on the launching stream (the cache is reset between sequences,
    # outside the events).  Reported: median (value) and minimum over the sequences.
    if warmup:
        free_run(warmup)
    for _ in range(max(args.warmup_sequences, 0)):
        free_run(steps)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    n_seq = max(args.sequences, 1)
    seq_ms = []
    for _ in range(n_seq):
        ctx.prefill_kv(kd, vd)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        edgefm_decode_step(handle, tok0, pos0, stream, None, None)
        for _ in range(steps - 1):
            edgefm_decode_step(handle, -1, -1, stream, None, None)
        e1.record()
        barrier()
        seq_ms.append(e0.elapsed_time(e1))

    # ---- end to end through the C ABI with host buffers: the token crosses PCIe both ways every step ----
    host_tok = torch.zeros(1, dtype=torch.int32).pin_memory()
    ctx.prefill_kv(kd, vd)
    barrier()
    t0 = time.perf_counter()
    tok, pos = tok0, pos0
    for _ in range(steps):
        edgefm_decode_step(handle, tok, pos, stream, None, ctx.next_token.data_ptr())   # request block: host -> device
        host_tok.copy_(ctx.next_token, non_blocking=True)                                # result: device -> host
        torch.cuda.current_stream().synchronize()
        tok, pos = int(host_tok[0]), pos + 1
    e2e_ms = (time.perf_counter() - t0) * 1e3
    clocks = sampler.stop()

    times = max_over_ranks(torch.tensor(seq_ms + [e2e_ms], dtype=torch.float64, device=dev), world)
    seq_ms, e2e_ms = [float(t) for t in times[:-1]], float(times[-1])
    launches = ctx.launches_per_step

    if rank == 0:
        tokens = steps * world
        ms_per_token, ms_per_token_min = per_token_stats(seq_ms, steps, world)
        dev_ms = ms_per_token * tokens                                   # median sequence time
        bytes_per_step = float(np.mean([cfg.step_bytes(cfg.cache_len + i) - (kv_saved_bytes(cfg, cfg.cache_len + i) if args.kv_format == "int8" else 0)
                                        for i in range(steps)])) - pruned_bytes
        gbs = bytes_per_step / (dev_ms / steps * 1e-3) / 1e9          # per GPU
        peak, peak_src = measured_peak()
        traffic, traffic_src = (None, None) if (n_sub or args.kv_format != "bf16") else ncu_traffic(cfg.name)
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
            cpu_ms = time_oracle(cfg, weights, k, v, args.cpu_steps, 1, args.kv_format)
            cpu = {"value": cpu_ms, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"{args.cpu_steps} full oracle decode steps at context {cfg.cache_len} (after 1 warm-up step)"
                             + ("; the oracle computes the whole output layer and restricts afterwards" if n_sub else "")}
        line = {
            "metric": METRIC, "value": ms_per_token, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": dev_ms / steps, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights/KV, fp32 accumulate" if args.kv_format == "bf16" else "bf16 weights, 8-bit KV codes with fp32 row scales, fp32 accumulate",
            "data": "synthetic",
            "config": config_block(cfg, workload, world, pruned_bytes),
            "timed_sequences": n_seq, "ms_per_token_min": ms_per_token_min,
            "tokens_per_s": tokens / (dev_ms * 1e-3),
            "roofline": {"bound": "hbm", "kernel": f"decode_megakernel: the whole decode step ({launches} kernel launch per token, one CUDA graph node)",
                         "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "peak_source": peak_src,
                         "bytes_per_launch": bytes_per_step, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "traffic": traffic, "traffic_source": traffic_src},
            "e2e": {"value": e2e_ms / tokens, "unit": UNIT, "h2d_bytes_per_step": 48, "d2h_bytes_per_step": 4},
            "gpu_launches": launches * steps * n_seq,
            "clocks": clocks,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
