#!/usr/bin/env python
"""Benchmark of the quantized Two-Branch Swin backbone forward (MixA-Q) on B200.

Metric: images/s of the Swin-T Two-Branch backbone at 800x1333 (200x334 tokens after the patch-4 stem),
W4 weights, A8 high / A4 low, as a function of the low-bit ratio; the headline `value` is at --ratio.
One "step" = one backbone forward of one synthetic image through the C ABI (mixaq_backbone_forward).

  python bench.py --gpus 1 --steps 20 --warmup 3                 # this library
  python bench.py --impl reference --steps 5 --warmup 1          # the CPU oracle, bounded sample per step
  torchrun --nproc-per-node N bench.py --gpus N ...              # N independent replicas (weak scaling)
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "swin_t_two_branch_backbone_images_per_sec_800x1333"
UNIT = "images/s"
SWEEP = [0.0, 0.25, 0.5, 0.75]                     # config 3 (the metric's axis)
SWEEP_BY_CONFIG = {3: SWEEP, 4: [0.0, 0.25, 0.5, 0.75], 5: [round(0.1 * i, 1) for i in range(9)]}   # config 5: 0 ... 0.8
L2_FLUSH_BYTES = 256 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 100 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
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
                p = [s.strip() for s in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); mx.append(float(p[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


CONFIG = 3          # --config: 3 = Swin-T 800x1333 (the metric's workload), 4 = Swin-S 1024^2 B=4, 5 = Swin-B 1536^2 B=2


def workload(ratio: float):
    from paper_2507_19131_b200 import synth
    if CONFIG == 4:
        wl = synth.config4()
        wl.low_ratios = [ratio] * len(wl.low_ratios)
        return wl
    if CONFIG == 5:
        return synth.config5(ratio=ratio)
    return synth.config3(ratio=ratio)


# ------------------------------------------------------------------------------------------------
# algorithmic work per kernel family for one backbone forward (used for the roofline of the dominant kernel)
# ------------------------------------------------------------------------------------------------
def algorithmic_work(wl, mq):
    """Returns {category: dict(ops=..., bytes=...)} for ONE forward.  Window-batch rows include Swin's pad
    tokens (the method computes them); MMA tile padding is excluded."""
    bb = wl.backbone
    B, H, W = wl.B, wl.H, wl.W
    work = {}

    def add(cat, ops=0.0, byt=0.0):
        w = work.setdefault(cat, dict(ops=0.0, bytes=0.0))
        w["ops"] += ops
        w["bytes"] += byt

    k = 0
    for s, (C, dep) in enumerate(zip(bb.dims, bb.depths)):
        if s > 0:
            Cp = bb.dims[s - 1]
            M = B * ((H + 1) // 2) * ((W + 1) // 2)
            bits = bb.merges[s - 1].aq.bits
            add("merge_gather_ln_quant", byt=B * H * W * Cp * 4 + M * 4 * Cp * bits / 8)
            add("gemm_merge", ops=2.0 * M * (4 * Cp) * (2 * Cp), byt=M * 4 * Cp * bits / 8 + M * 2 * Cp * 4)
            H, W = (H + 1) // 2, (W + 1) // 2
        add("energy", byt=B * H * W * (C * 4 + 4))
        for _ in range(dep):
            blk = bb.blocks[k]
            n_hi, n_lo, n_pr = mq.branch_counts(H, W, wl.low_ratios[k // 2], wl.prune_ratios[k // 2] if wl.prune_ratios else 0.0)
            Hd = blk.hidden
            for n, bits in ((n_hi, blk.hi.bits), (n_lo, blk.lo.bits)):
                M = B * n * 49
                cb = bits / 8.0
                add("gather_ln1_quant", byt=M * (C * 4 + C * cb))
                add("gemm_qkv", ops=2.0 * M * C * 3 * C, byt=M * (C * cb + 3 * C * cb))
                add("attention", ops=2.0 * M * 2 * 49 * C, byt=M * (3 * C * cb + C * cb))
                add("gemm_proj", ops=2.0 * M * C * C, byt=M * (C * cb + C * 4 + C * 4))
                add("ln2_quant", byt=M * (C * 4 + C * cb))
                add("gemm_fc1_gelu", ops=2.0 * M * C * Hd, byt=M * (C * cb + Hd * cb))
                work["gemm_fc1_gelu"]["alu_ops"] = work["gemm_fc1_gelu"].get("alu_ops", 0.0) + FC1_EPILOGUE_OPS * M * Hd
                add("gemm_fc2_scatter", ops=2.0 * M * Hd * C, byt=M * (Hd * cb + C * 4 + C * 4))
            add("select", byt=B * H * W * 4)
            add("copy_pruned", byt=B * n_pr * 49 * C * 8)
            k += 1
    return work


# The fc1 epilogue (zero-point correction, dequantize, GELU, quantize, pack) is a fixed sequence of binary32 / integer
# lane operations per output, set by the numeric contract (28 scalar operations); with K = C <= 768 the MMA needs
# K/64 <= 12 clocks per output row-chunk, so this family is bound by instruction issue, not by the tensor pipe.
FC1_EPILOGUE_OPS = 28
NUM_SMS = 148
TENSOR_CATS = {"gemm_qkv", "gemm_proj", "gemm_fc1_gelu", "gemm_fc2_scatter", "gemm_merge"}


def recorded_traffic(workload_name):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture) per kernel family of this
    workload, from profiles/ncu_dram_traffic.json; None when there is no record for the workload or the kernels have
    changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
    try:
        rec = json.load(open(path)).get(workload_name)
    except Exception:
        return None
    from paper_2507_19131_b200.ncu_summary import kernel_source_digest
    if not rec or rec.get("kernel_source_digest") != kernel_source_digest():
        return None
    return rec


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2507_19131_b200 import binding as mq
    from paper_2507_19131_b200 import replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    # a real (capturable) stream: on it the library replays each forward as one CUDA graph
    torch.cuda.set_stream(torch.cuda.Stream())
    ctx = mq.Context(local)
    K, Wm = args.steps, max(args.warmup, 3)
    # storage of the blocks' intermediate codes: bit-packed below this many channels, one code per byte from there on
    BYTE_MIN = args.byte_codes_min_dim if args.byte_codes_min_dim > 0 else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def time_ratio(ratio, steps, warm, sampler=None, e2e=False, byte_min="default"):
        byte_min = BYTE_MIN if byte_min == "default" else byte_min
        wl = workload(ratio)
        # replicas differ only in their seed-shifted input (weak scaling: one image per rank per step)
        x_host = torch.from_numpy(replicas.rank_input(wl.x, rank)).pin_memory()
        dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W, byte_codes_min_dim=byte_min)
        x_dev = x_host.cuda()
        outs_host = [torch.empty(o.shape, dtype=torch.float32).pin_memory() for o in dbb.outs]
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]

        def step():
            if e2e:
                x_dev.copy_(x_host, non_blocking=True)
            outs = mq.backbone_forward(ctx, dbb, x_dev, wl.low_ratios, wl.prune_ratios)
            if e2e:
                for h, o in zip(outs_host, outs):
                    h.copy_(o, non_blocking=True)

        for _ in range(warm):
            step()
        barrier()
        if sampler:
            sampler.start()
        t0 = time.perf_counter()
        for i in range(steps):
            flush.fill_(i & 0xFF)                    # evict L2 between timed iterations (outside the events)
            ev[i][0].record()
            step()
            ev[i][1].record()
        barrier()
        wall = time.perf_counter() - t0
        clocks = sampler.stop() if sampler else None
        ms = replicas.max_over_ranks(sum(a.elapsed_time(b) for a, b in ev), device="cuda")
        launches = ctx.launch_count()
        h2d = x_host.numel() * 4 if e2e else 0
        d2h = sum(h.numel() * 4 for h in outs_host) if e2e else 0
        return dict(ms=ms, wall=wall, clocks=clocks, launches=launches, h2d=h2d, d2h=d2h, wl=wl, dbb=dbb, x_dev=x_dev)

    def time_e2e(ratio, steps, warm):
        wl = workload(ratio)
        x_host = torch.from_numpy(replicas.rank_input(wl.x, rank)).pin_memory()
        comp = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        sets = []
        for _ in range(2):
            dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W, byte_codes_min_dim=BYTE_MIN)
            sets.append(dict(dbb=dbb, x=torch.empty_like(x_host, device="cuda"),
                             host=[torch.empty(o.shape, dtype=torch.float32).pin_memory() for o in dbb.outs],
                             e_in=torch.cuda.Event(), e_comp=torch.cuda.Event(), e_out=torch.cuda.Event()))
        torch.cuda.synchronize()

        def step(i):
            b = sets[i % 2]
            with torch.cuda.stream(s_in):
                s_in.wait_event(b["e_comp"])                 # the forward that last read this input buffer is done
                b["x"].copy_(x_host, non_blocking=True)
                b["e_in"].record(s_in)
            comp.wait_event(b["e_in"])
            comp.wait_event(b["e_out"])                      # the previous results of this set have left the device
            flush.fill_(i & 0xFF)
            outs = mq.backbone_forward(ctx, b["dbb"], b["x"], wl.low_ratios, wl.prune_ratios)
            b["e_comp"].record(comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["e_comp"])
                for h, o in zip(b["host"], outs):
                    h.copy_(o, non_blocking=True)
                b["e_out"].record(s_out)

        for i in range(warm + 2):
            step(i)
        barrier()
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_begin.record(comp)
        s_in.wait_event(t_begin); s_out.wait_event(t_begin)
        for i in range(steps):
            step(i)
        comp.wait_stream(s_out); comp.wait_stream(s_in)
        t_end.record(comp)
        barrier()
        ms = replicas.max_over_ranks(t_begin.elapsed_time(t_end), device="cuda")
        h2d, d2h = x_host.numel() * 4, sum(h.numel() * 4 for h in sets[0]["host"])

        # what the host link gives these very buffers, each direction alone (the pipeline cannot be faster than the
        # slower of the two): 5 copies each, CUDA events on the copying stream
        def link_gbs(stream, fn, nbytes, reps=5):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                fn()
                a.record(stream)
                for _ in range(reps):
                    fn()
                b_.record(stream)
            stream.synchronize()
            return nbytes * reps / (a.elapsed_time(b_) * 1e-3) / 1e9
        b0 = sets[0]
        up = link_gbs(s_in, lambda: b0["x"].copy_(x_host, non_blocking=True), h2d)
        down = link_gbs(s_out, lambda: [h.copy_(o, non_blocking=True) for h, o in zip(b0["host"], b0["dbb"].outs)], d2h)
        barrier()
        return dict(ms=ms, wl=wl, h2d=h2d, d2h=d2h, h2d_gbs=up, d2h_gbs=down)

    sampler = ClockSampler(local) if rank == 0 else None
    main = time_ratio(args.ratio, K, Wm, sampler)
    ms_per_step = main["ms"] / K
    value = replicas.job_throughput(wl_images(main["wl"]), K, world, main["ms"])

    # per-kernel CUDA-event breakdown: a separate pass of the same K steps with events around every kernel
    ctx.profile_begin()
    for _ in range(K):
        mq.backbone_forward(ctx, main["dbb"], main["x_dev"], main["wl"].low_ratios, main["wl"].prune_ratios)
    prof = ctx.profile_end()
    work = algorithmic_work(main["wl"], mq)
    kernels = {}
    # what an event pair adds by itself (pairs with nothing between them, recorded in the same graphs)
    b_ms, b_cnt = prof.pop("empty_event_bracket", (0.0, 0))
    bracket_ms = b_ms / b_cnt if b_cnt else 0.0
    for cat, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        w = work.get(cat, dict(ops=0.0, bytes=0.0))
        per_fwd_ms = ms / K
        kernels[cat] = dict(ms_per_step=round(per_fwd_ms, 5), launches_per_step=cnt // K,
                            share=0.0, tops=round(w["ops"] / (per_fwd_ms * 1e-3) / 1e12, 3) if w["ops"] else None,
                            gbs=round(w["bytes"] / (per_fwd_ms * 1e-3) / 1e9, 1),
                            ms_net_of_bracket=round(max(per_fwd_ms - bracket_ms * (cnt // K), 0.0), 5))
    tot = sum(v["ms_per_step"] for v in kernels.values()) or 1.0
    for v in kernels.values():
        v["share"] = round(v["ms_per_step"] / tot, 4)
    # Roofline: the path's contractions are the five GEMM families; their aggregate rate (useful int8 operations of one
    # forward over the summed CUDA-event time of the GEMM launches) against the int8 tensor peak = 2 x the measured bf16
    # peak (nominal int8 : bf16 ratio).  Each launch is bracketed by its own events, i.e. timed alone: the burst figure
    # is the denominator; the fraction against the sustained figure is given beside it.
    gemm_cats = [c for c in kernels if c in TENSOR_CATS]
    gemm_ms = sum(kernels[c]["ms_per_step"] for c in gemm_cats)
    gemm_ops = sum(work[c]["ops"] for c in gemm_cats)
    gemm_launches = sum(kernels[c]["launches_per_step"] for c in gemm_cats)
    peak_burst, peak_sust = 2.0 * peaks["bf16_burst"], 2.0 * peaks["bf16_sustained"]
    agg_tops = gemm_ops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    rec = recorded_traffic(main["wl"].name)
    traffic = None
    if rec:
        try:
            traffic = sum(rec["bytes_per_step"][c] for c in gemm_cats) / max(1, gemm_launches)
        except Exception:
            traffic = None
    dom = max(kernels, key=lambda c: kernels[c]["ms_per_step"])
    clk = (main["clocks"] or {}).get("sm_mhz") or 1965.0
    roof = dict(kernel="k_gemm_tc (QKV, proj, fc1+GELU, fc2+scatter, merge: all GEMM launches of one forward)",
                bound="tensor", achieved=round(agg_tops, 3), peak=round(peak_burst, 1), unit="TOP/s(int8)",
                frac=round(agg_tops / peak_burst, 5), frac_of_sustained=round(agg_tops / peak_sust, 5),
                peak_source=f"2 x bf16_tflops (burst) of {peaks['source']} peaks; sustained: 2 x bf16_tflops_sustained",
                launches_per_step=gemm_launches, launch_us=round(1e3 * gemm_ms / max(1, gemm_launches), 3),
                gemm_ms_per_step=round(gemm_ms, 5), gemm_gop_per_step=round(gemm_ops / 1e9, 2),
                event_bracket_us=round(bracket_ms * 1e3, 3),
                frac_net_of_bracket=round(gemm_ops / max((gemm_ms - bracket_ms * gemm_launches) * 1e-3, 1e-9) / 1e12 / peak_burst, 5),
                net_note=("every launch is timed between two event records, which by themselves take event_bracket_us "
                          "(pairs with nothing between them, same graphs); frac uses the bracketed times as they are, "
                          "frac_net_of_bracket subtracts that per launch.  Check: the net kernel times of one forward sum to "
                          f"{sum(v['ms_net_of_bracket'] for v in kernels.values()):.4f} ms against {ms_per_step:.4f} ms per timed forward"),
                traffic=traffic,
                traffic_note=("mean dram bytes per GEMM launch (ncu, profiles/ncu_dram_traffic.json)" if traffic is not None else
                              "no ncu record for these kernel sources and this workload"),
                per_family={c: dict(tops=kernels[c]["tops"], tensor_frac_burst=round(kernels[c]["tops"] / peak_burst, 5),
                                    tensor_frac_sustained=round(kernels[c]["tops"] / peak_sust, 5),
                                    ms_per_step=kernels[c]["ms_per_step"]) for c in gemm_cats},
                dominant_kernel=dom,
                timed="separate pass of K steps with CUDA events around every kernel, on the launching stream")
    if "gemm_fc1_gelu" in kernels:
        # what bounds the code-output epilogues: instruction issue.  Warp instructions per output come from the ncu
        # counter smsp__inst_executed of the recorded capture when there is one.
        fk = kernels["gemm_fc1_gelu"]
        outs = work["gemm_fc1_gelu"]["alu_ops"] / FC1_EPILOGUE_OPS
        issue_peak = NUM_SMS * 4 * clk * 1e6                    # warp instructions per second: 4 schedulers per SM
        note = dict(kernel="gemm_fc1_gelu", outputs_per_step=int(outs),
                    outputs_per_s=round(outs / (fk["ms_per_step"] * 1e-3) / 1e12, 4), unit="T outputs/s")
        wi = (rec or {}).get("fc1_warp_inst_per_32_outputs")
        if wi:
            note.update(warp_inst_per_32_outputs=wi,
                        issue_frac=round(outs / 32.0 * wi / (fk["ms_per_step"] * 1e-3) / issue_peak, 4),
                        issue_peak="148 SMs x 4 schedulers x sampled SM clock; instruction count from ncu smsp__inst_executed")
        roof["alu_note"] = note

    # end to end through the public call with HOST buffers (pinned): every step copies its image host->device, runs
    # the forward and copies the four stage maps device->host.  Two buffer sets and three streams let the copies of
    # neighbouring steps overlap the compute (PCIe is full duplex); the timed region is the whole pipeline of K steps.
    e2e = time_e2e(args.ratio, K, Wm)
    e2e_value = replicas.job_throughput(wl_images(e2e["wl"]), K, world, e2e["ms"])

    # the same forward with every block's codes bit-packed (what the expansion in shared memory costs in stages 3-4)
    packed_value = None
    if BYTE_MIN is not None and world == 1:
        n_p = max(3, K // 2)
        s_p = time_ratio(args.ratio, n_p, 3, byte_min=None)
        packed_value = round(wl_images(s_p["wl"]) * n_p / (s_p["ms"] / 1e3), 2)

    sweep = {}
    if args.sweep and world == 1:
        for r in SWEEP_BY_CONFIG[CONFIG]:
            if abs(r - args.ratio) < 1e-9:
                sweep[str(r)] = round(value, 2)
                continue
            s = time_ratio(r, max(3, K // 2), 3)
            sweep[str(r)] = round(wl_images(s["wl"]) * max(3, K // 2) / (s["ms"] / 1e3), 2)

    # the paper's axis: relative cost in bit operations (Appendix 6.2) of every swept ratio, with this shape's MACs
    from paper_2507_19131_b200 import cost_model as cm
    bbm = main["wl"].backbone
    pair_g, fixed_g = cm.backbone_pair_gmacs(bbm.dims, bbm.depths, main["wl"].H, main["wl"].W)
    cost = {str(r): {"relative_bops": round(cm.relative_cost([r] * len(pair_g), pair_g, fixed_g), 4),
                     "equivalent_act_bits": round(cm.equivalent_act_bits([r] * len(pair_g), float(bbm.blocks[0].hi.bits), pair_g, fixed_g), 3)}
            for r in (SWEEP_BY_CONFIG[CONFIG] if args.sweep else [args.ratio])}

    # the same forward with the steps on either side of the path inside the call and its graph: raw image ->
    # patch embedding -> two-branch backbone -> LayerNorm of the four stage maps (one mixaq_backbone_forward call)
    stem = None
    if CONFIG == 3 and world == 1:
        from paper_2507_19131_b200 import synth
        rng = np.random.default_rng(77)
        wl_s = main["wl"]
        emb = synth.make_embed(rng, bbm.dims[0])
        norms = [(np.ones(c, np.float32), np.zeros(c, np.float32)) for c in bbm.dims]
        dbs = mq.DeviceBackbone(ctx, wl_s.backbone, wl_s.B, 800, 1333, embed=emb, norms=norms, byte_codes_min_dim=BYTE_MIN)
        img = torch.from_numpy(synth.input_image(78, wl_s.B, 800, 1333)).cuda()
        for _ in range(3):
            mq.backbone_forward(ctx, dbs, img, wl_s.low_ratios, wl_s.prune_ratios)
        n_s = max(5, K)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_s)]
        for i in range(n_s):
            flush.fill_(i & 0xFF)
            evs[i][0].record()
            mq.backbone_forward(ctx, dbs, img, wl_s.low_ratios, wl_s.prune_ratios)
            evs[i][1].record()
        torch.cuda.synchronize()
        ms_s = sum(a.elapsed_time(b) for a, b in evs) / n_s
        stem = {"value": round(wl_s.B / (ms_s * 1e-3), 2), "unit": UNIT, "ms_per_step": round(ms_s, 4),
                "launches_per_step": ctx.launch_count(),
                "note": "800x1333x3 image -> patch embedding -> backbone -> LayerNorm of the 4 stage maps, one call, one graph"}

    # tensor-core issue rate as the library's own MMA loop reaches it (context for the tensor fractions above)
    mma_peak = None
    if world == 1:
        mma_peak = {"kind_i8_tops": round(ctx.measure_mma_peak(0, 8000), 1),
                    "kind_f8f6f4_e4m3_tops": round(ctx.measure_mma_peak(1, 8000), 1),
                    "kind_mxf4_e2m1_tops": round(ctx.measure_mma_peak(2, 8000), 1),
                    "note": "all SMs issue 128x256xK tcgen05.mma from shared memory into TMEM (K = 32; mxf4: K = 64 from the "
                            "same bytes).  f8f6f4 carries the 4/6-bit formats in 8-bit containers and is not faster than i8; "
                            "mxf4 is the block-scaled E2M1 path (grid 0, 1/2, 1, 3/2, 2, 3, 4, 6 and their negatives)"}

    status = ctx.device_status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    line = {
        "metric": METRIC if CONFIG == 3 else "two_branch_swin_backbone_images_per_sec_config%d" % CONFIG,
        "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8 MMA (int32 accumulate) + f32 epilogues", "data": "synthetic",
        "config": {"workload": main["wl"].name,
                   "dims": list(bbm.dims), "depths": list(bbm.depths),
                   "tokens": [main["wl"].H, main["wl"].W], "batch_per_gpu": main["wl"].B,
                   "weights": "W%d (int8 container)" % bbm.blocks[0].qkv.bits,
                   "act_bits_high_low": [bbm.blocks[0].hi.bits, bbm.blocks[0].lo.bits], "low_ratio": args.ratio,
                   "prune_ratio": (main["wl"].prune_ratios or [0.0])[0],
                   "code_storage": ("bit-packed in every block" if BYTE_MIN is None else
                                    f"bit-packed in blocks of fewer than {BYTE_MIN} channels, one code per byte from {BYTE_MIN} on"),
                   "l2": f"flushed between timed iterations ({L2_FLUSH_BYTES >> 20} MiB write)",
                   "parallelism": "replicas only (one image per GPU, no collective)"},
        "clocks": main["clocks"],
        "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": round(e2e["ms"] / K, 4),
                "pipeline": "2 buffer sets, copy-in / compute / copy-out streams; K steps timed as one pipeline",
                "host_link_gbs": {"h2d": round(e2e["h2d_gbs"], 2), "d2h": round(e2e["d2h_gbs"], 2)},
                "link_bound_ms_per_step": round(max(e2e["h2d"] / e2e["h2d_gbs"], e2e["d2h"] / e2e["d2h_gbs"]) / 1e6, 4),
                "note": "the four binary32 stage maps leave the device every step; when link_bound_ms_per_step exceeds "
                        "ms_per_step of the resident run, the end-to-end figure is set by this host's PCIe link, not by the kernels"},
        "gpu_launches": main["launches"] * K,
        "roofline": roof,
        "kernels": kernels,
        "value_all_bit_packed": packed_value,
        "low_ratio_sweep_images_per_sec": sweep,
        "paper_cost_model": cost,
        "value_with_stem": stem,
        "mma_issue_rate": mma_peak,
        "device_status": status,
    }
    if args.cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(full=True)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def wl_images(wl):
    return wl.B


# ------------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# ------------------------------------------------------------------------------------------------
def oracle_sample(crop_h: int, crop_w: int, ratio: float):
    """Times the oracle (as it stands) on a crop of the workload; returns (seconds, images-equivalent, threads)."""
    from oracle import oracle as orc
    wl = workload(ratio)
    x = np.ascontiguousarray(wl.x[:, :crop_h, :crop_w])
    t0 = time.perf_counter()
    orc.backbone_forward(wl.backbone, x, wl.low_ratios, wl.prune_ratios)
    dt = time.perf_counter() - t0
    frac = (crop_h * crop_w) / float(wl.H * wl.W)
    return dt, frac * wl.B, orc.get_threads(), wl


def cpu_baseline(full: bool, ratio: float = 0.5):
    from oracle import oracle as orc
    if full and CONFIG == 3:
        dt, imgs, thr, wl = oracle_sample(200, 334, ratio)
        sample = "one full forward of the same workload (1 image, 200x334 tokens)"
    else:
        dt, imgs, thr, wl = oracle_sample(50, 84, ratio)
        sample = "one forward of a 50x84-token crop of the workload's images, scaled by token count"
    out = {"value": round(imgs / dt, 5), "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample,
           "seconds": round(dt, 3)}
    # the same oracle on ONE thread, on the crop (the full image would take a minute)
    n = orc.get_threads()
    orc.set_threads(1)
    dt1, imgs1, _, _ = oracle_sample(50, 84, ratio)
    orc.set_threads(n)
    out["single_thread"] = {"value": round(imgs1 / dt1, 5), "cores": 1, "seconds": round(dt1, 3),
                            "sample": "50x84-token crop, scaled by token count"}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, Wm = args.steps, args.warmup
    from oracle import oracle as orc
    from paper_2507_19131_b200 import cost_model as cm
    wl = workload(args.ratio)
    bb = wl.backbone
    thr = orc.get_threads()
    # One untimed oracle forward, block by block, keeps every block's true input (and its stage's energy map).
    # A timed step then re-runs ONE block of the full-size workload (with the patch merging in front of it when it
    # opens a stage), cycling through the blocks; a full cycle is exactly one forward's work.  A step counts as the
    # block's share of the forward's multiply-accumulates.  (Spatial crops would leave most host cores idle in the
    # late stages, and every crop would still run all blocks.)
    pair_g, fixed_g = cm.backbone_pair_gmacs(bb.dims, bb.depths, wl.H, wl.W)
    work = []                                    # (share of the forward, callable)
    x, k, pair = wl.x, 0, 0
    total_g = sum(pair_g) + fixed_g
    H_, W_ = wl.H, wl.W
    for s_i, d in enumerate(bb.depths):
        pre = None
        if s_i > 0:
            m, x_in = bb.merges[s_i - 1], x
            mg = ((H_ + 1) // 2) * ((W_ + 1) // 2) * (4 * bb.dims[s_i - 1]) * (2 * bb.dims[s_i - 1]) * wl.B / 1e9
            pre = (mg / wl.B, (lambda m=m, x_in=x_in: orc.merge_forward(m, x_in)))
            x = orc.merge_forward(m, x)
            H_, W_ = (H_ + 1) // 2, (W_ + 1) // 2
        e = orc.energy(x, bb.blocks[k].score_inv_scale)
        lmax = pmax = 0.0
        for i in range(d):
            blk, x_in = bb.blocks[k], x
            lr = wl.low_ratios[k // 2]
            pr = wl.prune_ratios[k // 2] if wl.prune_ratios else 0.0
            lmax, pmax = max(lmax, lr), max(pmax, pr)
            share = pair_g[k // 2] / min(2, d)
            fn = (lambda blk=blk, x_in=x_in, e=e, lr=lmax, pr=pmax: orc.block_forward(blk, x_in, lr, pr, energy_map=e).y)
            if pre is not None and i == 0:
                share += pre[0]
                fn = (lambda f=fn, g=pre[1]: (g(), f())[1])
            work.append((share / total_g, fn))
            x = orc.block_forward(blk, x, lmax, pmax, energy_map=e).y
            k += 1
    for i in range(Wm):
        work[i % len(work)][1]()
    t0 = time.perf_counter()
    imgs = 0.0
    for i in range(K):
        share, fn = work[i % len(work)]
        fn()
        imgs += share * wl.B
    total = time.perf_counter() - t0
    value = imgs / total
    sample = ("each step = one block of the full-size workload on its true input (with the patch merging in front of "
              "it when it opens a stage), cycling through the %d blocks; counted as its share of the forward's MACs" % len(work))
    line = {
        "impl": "reference", "metric": METRIC if CONFIG == 3 else "two_branch_swin_backbone_images_per_sec_config%d" % CONFIG,
        "value": round(value, 5), "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": Wm, "ms_per_step": round(1e3 * total / K, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32/int64 integer + f32", "data": "synthetic",
        "config": {"workload": wl.name, "low_ratio": args.ratio, "sample": sample},
        "cpu_baseline": {"value": round(value, 5), "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 5), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ratio", type=float, default=0.5)
    ap.add_argument("--config", type=int, default=3, choices=[3, 4, 5],
                    help="3: Swin-T 800x1333 B=1 (the metric's workload); 4: Swin-S 1024^2 B=4 A4/A2 + 20 %% pruned; 5: Swin-B 1536^2 B=2")
    ap.add_argument("--no-sweep", dest="sweep", action="store_false")
    ap.add_argument("--sweep", dest="force_sweep", action="store_true",
                    help="also sweep the low-bit ratio for --config 4 (0 ... 0.75) or 5 (0 ... 0.8); config 3 sweeps by default")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--byte-codes-min-dim", type=int, default=384,
                    help="blocks with at least this many channels store their intermediate codes one per byte "
                         "(mixaq_block_params.byte_codes); 0: every block bit-packs")
    args = ap.parse_args()
    global CONFIG
    CONFIG = args.config
    if CONFIG != 3:
        args.sweep = bool(args.force_sweep)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
