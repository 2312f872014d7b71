#!/usr/bin/env python
"""Throughput of the token-wise RNN-T beam search (decoded encoder frames per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--segment 3] [--impl ours|reference]

One step = one tw_decode of the whole synthetic batch: every pass of Algorithm 1's inner loop (joiner
over the segment, softmax, Eq. 3-7, AddAndMerge, threshold, N-best expansions, predictor update) for
every utterance, plus the once-per-decode encoder projection.  Prints ONE JSON line.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import tw_synth  # noqa: E402

METRIC = "decoded frames/s at N=10,S=3 on 1 B200; joiner+expansion % of roofline"
UNIT = "frames/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(tw_synth.CONFIGS))
    ap.add_argument("--segment", type=int, default=0, help="segment size S (0: the workload's headline value)")
    ap.add_argument("--mode", default="auto", choices=["auto", "f32", "bf16"])
    ap.add_argument("--batch", type=int, default=0, help="utterances per GPU (0: the workload's batch)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lanes", action="store_true", help="decode the batch in one piece instead of two concurrent halves")
    ap.add_argument("--no-fused", action="store_true", help="bf16 mode: staged joiner kernels instead of the fused one")
    ap.add_argument("--monotonic", action="store_true", help="the monotonic RNN-T variant (every output consumes a frame)")
    ap.add_argument("--cpu-frames", type=int, default=0, help="frames of the CPU-baseline sample (0: auto)")
    ap.add_argument("--blank-threshold", type=float, default=None,
                    help="blank thresholding for a workload with the factorised output (h1): skip the label part of a "
                         "(hypothesis, frame) whose blank probability exceeds this")
    ap.add_argument("--no-largest", action="store_true", help="skip the fused kernel's leg at the largest step shape")
    ap.add_argument("--agreement-utterances", type=int, default=4, help="utterances of the bf16 top-1 agreement check (0: skip)")
    return ap.parse_args()


# DRAM traffic of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum per launch) from ncu captures
# of this same kernel: "cold" with the caches flushed before the launch (ncu's default), "warm" with the caches as
# the running decode leaves them (--cache-control none); the commands are in profiles/.  Each
# entry carries the digest of the kernel's sources at the time of the capture; once the sources differ the
# counters no longer describe the kernel that runs and the bench reports null.
KERNEL_SOURCES = ("fused_joiner.cu", "fused_joiner_kernel.inc", "fused_joiner_host.inc", "sm100.cuh")
NCU_DRAM_BYTES_PER_LAUNCH = {
    # (workload, S): (source digest, cold bytes, warm bytes)
    ("c3", 3): ("ee4da9199c29", 16897000, 14662000),      # cold: W_out + the A operand; warm: 2.0 MB read, 12.6 MB of delta_nb leaving L2
}


def kernel_source_digest():
    import hashlib
    h = hashlib.sha1()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2302_14357_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def ncu_traffic(workload, S):
    ent = NCU_DRAM_BYTES_PER_LAUNCH.get((workload, S))
    if ent is None or ent[0] != kernel_source_digest():
        return None, None
    return {"cold": ent[1], "warm": ent[2]}, ent[0]


def joiner_kernel_name(mode_name, st):
    if mode_name == "bf16" and st.get("fused_on"):
        return "fused_joiner_kernel (contraction + softmax + Eq. 3-7, tcgen05, cluster of V/256 CTAs)"
    if mode_name == "bf16":
        return "gemm_bf16_kernel (joiner contraction, tcgen05; logits to device memory)"
    return "gemm_f32_kernel<1> (joiner contraction, SIMT fp32)"


def headline_S(cfg):
    return 3 if 3 in cfg.S_values else cfg.S_values[0]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "tflops_burst": d["bf16_tflops"],
                "tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample of the same workload
def oracle_sample(cfg, S, frames, utt=0, monotonic=False, blank_threshold=None):
    from oracle import rnnt_model as rm
    from oracle import token_wise_search as tws
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg, batch=utt + 1)
    om = rm.RnntModel(m.W_e, m.W_p, m.W_out, m.b_out, m.emb, m.lstm_W_ih, m.lstm_W_hh, m.lstm_b,
                      activation=cfg.joiner_act, normalisation=cfg.joiner_norm)
    n = int(min(frames, lens[utt]))
    t0 = time.perf_counter()
    _, st = tws.token_wise_beam_search(om, enc[utt, :n], cfg.N, S, max_iters=4 * S + 16, monotonic=monotonic,
                                       blank_threshold=blank_threshold)
    dt = time.perf_counter() - t0
    return {"value": n / dt, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": "utterance %d of workload %s, first %d frames, N=%d S=%d, fp64 numpy; %.1f s"
                      % (utt, cfg.name, n, cfg.N, S, dt),
            "calls_per_frame": st.calls / max(n, 1), "joins_per_frame": st.joins / max(n, 1)}, dt


def top1_agreement(dec, cfg, S, enc_np, len_np, utterances, frames, monotonic=False, blank_threshold=None):
    """bf16 mode against the fp64 oracle: both decode the first `frames` frames of a few utterances of the
    bench batch; reports how often the best token sequence is the same and the largest score gap where it is."""
    from oracle import rnnt_model as rm
    from oracle import token_wise_search as tws
    K = int(min(utterances, enc_np.shape[0]))
    F = int(min(frames, enc_np.shape[1]))
    enc = np.ascontiguousarray(enc_np[:K, :F])
    lens = np.minimum(len_np[:K], F).astype(np.int32)
    tokens, olens, scores, status, _ = dec.decode(enc, lens)
    tokens, olens, scores = tokens.cpu().numpy(), olens.cpu().numpy(), scores.cpu().numpy()
    m = tw_synth.make_model(cfg)
    om = rm.RnntModel(m.W_e, m.W_p, m.W_out, m.b_out, m.emb, m.lstm_W_ih, m.lstm_W_hh, m.lstm_b,
                      activation=cfg.joiner_act, normalisation=cfg.joiner_norm)
    agree, gap = 0, 0.0
    for b in range(K):
        ref, _ = tws.token_wise_beam_search(om, enc[b, :lens[b]], cfg.N, S, max_iters=4 * S + 16, monotonic=monotonic,
                                            blank_threshold=blank_threshold)
        got = tuple(int(x) for x in tokens[b, 0, :max(int(olens[b, 0]), 0)])
        if got == ref[0][0]:
            agree += 1
            gap = max(gap, abs(float(scores[b, 0]) - ref[0][1]))
    return {"rate": agree / max(K, 1), "utterances": K, "frames_each": F, "max_score_gap": gap,
            "against": "fp64 oracle on the same bf16-rounded weights and frames"}


def largest_step_roofline(peaks, launches=20, warm=5):
    """The fused joiner kernel alone at the largest step shape of the workloads: B = 512 utterances x N = 10
    hypotheses x S = 10 frames = 51,200 joiner rows, V = 4096, J = 1024 (workload c4's model), timed with CUDA
    events around the kernel (tw_set_profiling) through tw_joiner_expand.  Operand (105 MB) and delta_nb (84 MB)
    exceed L2."""
    import torch
    from paper_2302_14357_b200.binding import MODE_BF16, TwDecoder, weights_from_synth
    cfg = tw_synth.get_config("c4")
    S, N, B = 10, cfg.N, cfg.batch
    R = B * N
    dec = TwDecoder(weights_from_synth(tw_synth.make_model(cfg)), N=N, S=S, mode=MODE_BF16, max_batch=B, max_T=2 * S)
    if not dec.set_fused(True):
        return None
    g = torch.Generator(device="cuda").manual_seed(4)
    E = torch.randn((B, S, cfg.J), device="cuda", generator=g)
    Pp = torch.randn((R, cfg.J), device="cuda", generator=g) * 0.5
    row_group = (torch.arange(R, device="cuda", dtype=torch.int32) // N).contiguous()
    ld_old = torch.randn((R, S), device="cuda", generator=g) - 2.0
    for _ in range(warm):
        dec.joiner_expand(E, Pp, row_group, None, ld_old)
    dec.set_profiling(True)
    for _ in range(launches):
        dec.joiner_expand(E, Pp, row_group, None, ld_old)
    st = dec.stats()
    dec.set_profiling(False)
    dec.close()
    if st["joiner_launches"] <= 0 or st["ns_joiner"] <= 0:
        return None
    us = st["ns_joiner"] * 1e-3 / st["joiner_launches"]
    flops = 2.0 * cfg.J * cfg.V * R * S
    achieved = flops / (us * 1e-6) / 1e12
    return {"workload": "c4-step (R=%d rows x S=%d frames, V=%d, J=%d)" % (R, S, cfg.V, cfg.J),
            "kernel": "fused_joiner_kernel", "bound": "tensor", "achieved": achieved, "unit": "TFLOP/s",
            "peak": peaks["tflops_sustained"], "frac": achieved / peaks["tflops_sustained"],
            "frac_burst": achieved / peaks["tflops_burst"], "avg_launch_us": us, "launches": int(st["joiner_launches"]),
            "flops_per_launch": flops, "operand_kernel_avg_us": st["ns_scan"] * 1e-3 / st["joiner_launches"]}


def auto_cpu_frames(cfg):
    # sized for roughly 10-30 s of oracle time on a few host cores
    cost = cfg.J * cfg.V * cfg.N / (640 * 1024 * 10)
    return int(max(24, min(cfg.T, 600, 4000 / max(cost, 0.05))))


def run_reference(args, cfg, S):
    """The reference arm: the fp64 oracle on host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    frames = args.cpu_frames or max(12, auto_cpu_frames(cfg) // 4)
    for _ in range(args.warmup):
        oracle_sample(cfg, S, max(4, frames // 4), monotonic=args.monotonic, blank_threshold=args.blank_threshold)
    times, vals, last = [], [], None
    for k in range(args.steps):
        last, dt = oracle_sample(cfg, S, frames, utt=0, monotonic=args.monotonic, blank_threshold=args.blank_threshold)
        times.append(dt)
        vals.append(last["value"])
    value = frames * len(times) / sum(times) if times else 0.0
    base = dict(last or {})
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / max(len(times), 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "N": cfg.N, "S": S, "sample_frames_per_step": frames,
                       "variant": "monotonic" if args.monotonic else "standard"},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(device_index), "--query-gpu=" + self.QUERY,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
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
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def run_ours(args, cfg, S):
    import torch
    import torch.distributed as dist
    from paper_2302_14357_b200.binding import MODE_BF16, MODE_F32, TwDecoder, weights_from_synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the decoder has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    mode_name = cfg.dtype if args.mode == "auto" else args.mode
    mode = MODE_BF16 if mode_name == "bf16" else MODE_F32
    B = args.batch or cfg.batch
    model = tw_synth.make_model(cfg)
    # every rank decodes its own batch of the same shape (utterances are independent: no exchange)
    enc_np, len_np = tw_synth.make_encoder_batch(cfg.with_(seed=cfg.seed + 1000 * rank), batch=B)
    # a bf16 workload crosses the boundary as bf16 (tw_model::dtype): weights and encoder frames in 2 bytes per element
    io_dtype = "bf16" if cfg.dtype == "bf16" else "f32"
    tdt = torch.bfloat16 if io_dtype == "bf16" else torch.float32
    dec = TwDecoder(weights_from_synth(model), N=cfg.N, S=S, mode=mode, max_batch=B, max_T=cfg.T, joiner_act=cfg.joiner_act,
                    dtype=io_dtype)
    if args.no_fused:
        dec.set_fused(False)
    if args.no_lanes:
        dec.set_lanes(False)
    if args.monotonic:
        dec.set_monotonic(True)
    if args.blank_threshold is not None and dec.set_blank_threshold(args.blank_threshold) != 0:
        raise RuntimeError("--blank-threshold needs a workload with the factorised output (h1) and a value in [0, 1]")
    enc = torch.from_numpy(enc_np).to(tdt).cuda()       # exact: the workload's frames are bf16-representable
    lens = torch.from_numpy(len_np).cuda()
    frames = int(len_np.sum())

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # L2 hygiene: a workload whose inputs do not exceed L2 (126 MB) several times over gets L2 flushed
    # (a 256 MB write) before every timed step, outside the timed interval
    flush = None if enc.numel() * enc.element_size() > 3 * 126e6 else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    def timed(fn, steps):
        barrier()
        pairs = []
        for _ in range(steps):
            if flush is not None:
                flush.zero_()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            fn()                      # synchronous: tw_decode returns after its stream has drained
            ev1.record()
            pairs.append((ev0, ev1))
        barrier()
        ms = sum(a.elapsed_time(b) for a, b in pairs)
        if world > 1:
            t = torch.tensor([ms], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    for _ in range(args.warmup):
        dec.decode(enc, lens)
    # device-resident inputs: the timed region holds only tw_decode calls
    sampler = ClockSampler(local) if rank == 0 else None
    ms = timed(lambda: dec.decode(enc, lens), args.steps)
    # the same K decodes again with per-stage CUDA events on the decode stream (about four event records
    # per device step, which cost a few percent to 20 % on the latency-bound workloads): stage shares and
    # the dominant kernel's launch durations come from this pass, the headline value from the one above
    dec.set_profiling(True)
    ms_profiled = timed(lambda: dec.decode(enc, lens), args.steps)
    clocks = sampler.stop() if sampler else None
    st = dec.stats()            # of the last profiled decode (every decode does identical work)
    dec.set_profiling(False)

    # end to end: pinned host buffers in, host buffers out, copies inside the timed region
    enc_pin = torch.from_numpy(enc_np).to(tdt).contiguous().pin_memory()
    len_pin = torch.from_numpy(len_np).pin_memory()
    outs = (torch.empty((B, cfg.N, dec.U_cap), dtype=torch.int32).pin_memory().numpy(),
            torch.empty((B, cfg.N), dtype=torch.int32).pin_memory().numpy(),
            torch.empty((B, cfg.N), dtype=torch.float64).pin_memory().numpy(),
            torch.empty((B,), dtype=torch.int32).pin_memory().numpy())
    e2e_steps = max(1, min(args.steps, 3))
    dec.decode_host(enc_pin, len_pin.numpy(), out=outs)
    ms_e2e = timed(lambda: dec.decode_host(enc_pin, len_pin.numpy(), out=outs), e2e_steps)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    value = world * frames * args.steps / (ms * 1e-3)
    e2e_value = world * frames * e2e_steps / (ms_e2e * 1e-3)
    # dominant kernel: the joiner contraction, 2*J*V flops per (row, frame)
    flops_per_row = 2.0 * cfg.J * cfg.V
    joiner_s = st["ns_joiner"] * 1e-9
    achieved = st["joiner_frame_rows"] * flops_per_row / joiner_s / 1e12 if joiner_s > 0 else 0.0
    peak = peaks["tflops_sustained"]
    stage_ns = {k: st[k] for k in ("ns_prologue", "ns_predictor", "ns_joiner", "ns_scan", "ns_hyp")}
    tot_ns = max(1, sum(stage_ns.values()))
    traffic, traffic_rev = ncu_traffic(cfg.name, S) if (mode_name == "bf16" and st.get("fused_on")) else (None, None)
    # the HBM-side kernels of a step, from the same stage events: algorithmic bytes per decode / device time
    fused = mode_name == "bf16" and st.get("fused_on")
    hbm = {}
    if fused and st["steps"] > 0:
        rows, frame_rows, steps = st["rows"], st["joiner_frame_rows"], st["steps"]
        # hyp_step_kernel: every row's delta_nb [V] float32 read once (selection) + per row about 64 B of list state
        b_hyp = rows * (4.0 * dec.Vp + 64.0)
        # operand kernel: E rows (float32) and Pp rows (float32) read, act(E + Pp) written as bf16
        b_op = frame_rows * cfg.J * (4.0 + 2.0) + rows * cfg.J * 4.0
        for name, nbytes, ns in (("hyp_step_kernel (selection over delta_nb, AddAndMerge, threshold, new list A)", b_hyp, st["ns_hyp"]),
                                 ("joiner_A_tiled_kernel (operand act(E + Pp) as bf16)", b_op, st["ns_scan"])):
            if ns > 0:
                gbs = nbytes / (ns * 1e-9) / 1e9
                hbm[name.split(" ")[0]] = {"kernel": name, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                           "frac": gbs / peaks["hbm_gbs"], "avg_launch_us": ns * 1e-3 / steps,
                                           "bytes_per_launch": nbytes / steps}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "ms_per_step_with_stage_events": ms_profiled / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": mode_name, "data": "synthetic",
        "config": {"workload": cfg.name, "B_per_gpu": B, "T": cfg.T, "N": cfg.N, "S": S, "J": cfg.J, "V": cfg.V,
                   "mode": mode_name, "boundary_dtype": io_dtype, "variant": "monotonic" if args.monotonic else "standard", "joiner_norm": cfg.joiner_norm,
                   "blank_threshold": args.blank_threshold, "l2": ("inputs larger than L2 (encoder batch %.0f MB)" % (enc.numel() * enc.element_size() / 1e6)) if flush is None
                         else "L2 flushed by a 256 MB write before every timed step (encoder batch %.0f MB)" % (enc.numel() * enc.element_size() / 1e6),
                   "parallelism": "independent utterance batches per GPU, no collective"},
        "calls_per_frame": st["calls"] / max(st["frames"], 1), "joins_per_frame": st["joins"] / max(st["frames"], 1),
        "device_steps_per_decode": st["steps"], "avg_rows_per_step": st["rows"] / max(st["steps"], 1),
        "limit_hits": st["limit_hits"], "frame_rows_skipped_share": st["frame_rows_skipped"] / max(st["joiner_frame_rows"], 1),
        "stage_share": {k[3:]: round(v / tot_ns, 4) for k, v in stage_ns.items()},
        "stage_ms_per_decode": {k[3:]: round(v * 1e-6, 3) for k, v in stage_ns.items()},
        "roofline": {"kernel": joiner_kernel_name(mode_name, st), "bound": "tensor", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak if peak else None,
                     "frac_sustained": achieved / peaks["tflops_sustained"], "frac_burst": achieved / peaks["tflops_burst"],
                     "peak_burst": peaks["tflops_burst"],
                     # bytes per launch: the ncu capture with the caches flushed before the launch (the profiling
                     # recipe's); traffic_warm: with the caches as the running decode leaves them
                     "traffic": traffic["cold"] if traffic else None,
                     "traffic_warm": traffic["warm"] if traffic else None, "traffic_kernel_digest": traffic_rev,
                     "peak_source": "%s bf16 sustained (a seconds-long cuBLAS loop under the power cap); frac_burst is against the "
                                    "burst figure, measured at the SM clock in `clocks`" % peaks["source"],
                     "avg_launch_us": 1e6 * joiner_s / max(st["joiner_launches"], 1),
                     "flops_per_launch": st["joiner_frame_rows"] * flops_per_row / max(st["joiner_launches"], 1)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(enc_pin.numel() * enc_pin.element_size() + len_np.nbytes),
                "d2h_bytes_per_step": int(sum(o.nbytes for o in outs))},
        "gpu_launches": int(st["kernel_launches"] * args.steps),
        "clocks": clocks,
    }
    if hbm:
        line["roofline_hbm"] = hbm
    if mode_name == "bf16" and world == 1 and not args.no_largest:
        big = largest_step_roofline(peaks)
        if big is not None:
            line["roofline_largest"] = big
    if mode_name == "bf16" and world == 1 and not args.no_cpu_baseline and args.agreement_utterances > 0:
        line["bf16_top1_agreement"] = top1_agreement(dec, cfg, S, enc_np, len_np, args.agreement_utterances,
                                                     min(150, args.cpu_frames or auto_cpu_frames(cfg)), args.monotonic, args.blank_threshold)
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"], _ = oracle_sample(cfg, S, args.cpu_frames or auto_cpu_frames(cfg), monotonic=args.monotonic,
                                                 blank_threshold=args.blank_threshold)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    cfg = tw_synth.get_config(args.workload)
    S = args.segment or headline_S(cfg)
    if args.impl == "reference":
        run_reference(args, cfg, S)
    else:
        run_ours(args, cfg, S)


if __name__ == "__main__":
    main()
