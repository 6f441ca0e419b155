#!/usr/bin/env python
"""Throughput benchmark of the integer-flow encoder on B200.

One step = one encode (all levels: squeeze, couplings, split, prior heads) of one batch of the
ImageNet64-shaped pruned flow (batch 128 of uint8 3x64x64 synthetic smooth-field images, 4 levels
x 8 couplings, hidden 256 with 30-60 % of the filters pruned). Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 2] [--batch B]

With N > 1 (launched by torch.distributed.run) every rank encodes its own batch (weak scaling,
no collective on the data path); the time is the maximum over ranks.
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import iodf_synth as S

METRIC = "flow_encode_images_per_sec"
UNIT = "images/s"
N_SETS = 8   # rotating input/output sets: 8 x 19.7 MB > the 126 MB L2


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d["hbm_gbs"], d["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def kernel_sources_hash(names):
    """SHA-256 of the named kernel sources: ties a stored profiler counter to the code it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2206_08869_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def stored_traffic(key):
    """DRAM bytes per launch of the dominant kernel from the committed profiler capture, or None
    (with the reason) when there is no capture for this workload or the kernel has changed since."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None, "no capture stored"
    with open(p) as f:
        d = json.load(f)
    e = d.get(key)
    if e is None:
        return None, "no capture for " + key
    if e.get("sources_sha256") != kernel_sources_hash(e.get("sources", [])):
        return None, "kernel sources changed since the capture"
    return float(e["dram_bytes_per_launch"]), e.get("capture", "")


def measure_int8_peak(G, m, stream, torch):
    """TOP/s of the MMA-only kernel: best single launch of ~10 ms (burst) and ~1 s of launches back to
    back (sustained), CUDA events on the launching stream."""
    G.iodf_int8_mma_peak(m, 4000, stream)
    stream.synchronize()

    def run(groups, launches):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ops = 0
        for _ in range(launches):
            ops += G.iodf_int8_mma_peak(m, groups, stream)
        b.record(stream)
        b.synchronize()
        return ops / (a.elapsed_time(b) * 1e-3) / 1e12
    groups = 20000                       # 160 000 MMAs per SM: about 10 ms
    burst = max(run(groups, 1) for _ in range(3))
    sustained = run(groups, 100)
    G.iodf_check(m)
    return burst, sustained


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.sm, self.reasons, self.max_sm = index, False, [], set(), None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                     nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                     nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                     nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
            while not self.stop_flag:
                self.sm.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, nm in names.items():
                    if r & bit:
                        self.reasons.add(nm)
                time.sleep(0.01)
        except Exception as e:  # NVML unavailable: report that instead of clocks
            self.reasons.add("nvml_error:%s" % type(e).__name__)

    def summary(self):
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_sm,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def oracle_rate(model, cfg, batch, cores, seconds=0.0):
    """images/s of the CPU oracle on a bounded sample of the workload: max(cores, 16) images, or, with
    `seconds`, as many (a multiple of the cores, at most 1024) as that first sample says fill the time."""
    import oracle as O
    pk = O.Packed(model)

    def run(n):
        x = S.config_images(cfg, batch=n)
        t0 = time.perf_counter()
        O.forward(pk, x, threads=cores)
        return time.perf_counter() - t0
    n = max(cores, 16)
    dt = run(n)
    more = int(min(1024, seconds * n / dt)) // cores * cores
    if more > n:
        n = more
        dt = run(n)
    return n / dt, n, dt


def run_reference(args, rank):
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    model = S.config_model(args.config)
    rates = []
    for i in range(args.warmup + args.steps):
        r, n, dt = oracle_rate(model, args.config, args.batch, cores)
        if i >= args.warmup:
            rates.append((r, dt))
    value = float(np.mean([r for r, _ in rates]))
    sample = "%d images of the workload per step, oracle forward, %d threads" % (n, cores)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean([d for _, d in rates])),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": workload(args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def max_over_ranks(values, world, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity for one rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(images_per_rank_per_step, world, steps, seconds):
    """Whole-job images/s: every rank processes its own batch, the slowest rank sets the time."""
    return images_per_rank_per_step * world * steps / seconds


def rank_seed_offset(rank, i):
    """Distinct synthetic input sets per rank and per rotating buffer."""
    return 100 * rank + i


def workload(args):
    c = S.CONFIGS[args.config]
    net = ", %d residual blocks per coupling" % c["n_blocks"] if c.get("n_blocks") else ""
    return {"workload": "config %s: ImageNet%d-shaped pruned IODF encode, batch %d of uint8 3x%dx%d, %d levels x %d "
                        "couplings, hidden %d%s" % (args.config, c["hw"], args.batch, c["hw"], c["hw"],
                                                     len(c["splits"]), c["n_couplings"], c["hidden"], net),
            "batch_per_gpu": args.batch, "l2_policy": "rotating %d input/output sets (> L2)" % N_SETS,
            "parallelism": "independent batches per GPU, no collective"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200")
    ap.add_argument("--config", default="2")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--in-flight", type=int, default=4, help="steps in flight at the same time (streams); 1 = one after the other")
    args = ap.parse_args()
    args.config = int(args.config) if args.config.isdigit() else args.config
    args.batch = args.batch or S.CONFIGS[args.config]["batch"]
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2206_08869_b200 as G

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg, B = args.config, args.batch
    model = S.config_model(cfg)
    m = G.iodf_create(model, B, device=local_rank)
    lay = m.layout
    macs = int(lay.macs_per_image)

    xs = [torch.from_numpy(S.config_images(cfg, batch=B, seed_offset=rank_seed_offset(rank, i))).to(dev) for i in range(N_SETS)]
    zs = [torch.empty((B, m.d), dtype=torch.int32, device=dev) for _ in range(N_SETS)]
    ps = [torch.empty((B, 2, m.d_fact), dtype=torch.int32, device=dev) for _ in range(N_SETS)]
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput ----------------------------------------------------------
    # Blocks of `steps` back-to-back encodes, each block between two events; the blocks repeat until
    # the timed region is at least 0.25 s (so that the clock sampler sees it whatever `steps` is).
    # ms_per_step is the median block; the minimum is reported beside it.
    # `--in-flight F` steps run at the same time, each on a stream and a model handle of its own (the
    # sets of a step's inputs and outputs rotate over N_SETS > F, so steps in flight never share one).
    # A level's launch is one CTA per image; with several steps in flight the SMs that a batch of 128
    # leaves idle, and the ends of every level, are filled by the neighbouring steps.
    F = max(1, min(int(args.in_flight), N_SETS - 1))
    # Handles of steps in flight are made with the throughput plan (fewer CTAs per launch at the deep
    # levels); `m`, the handle of everything timed one call at a time, with the default plan.
    lanes = [(m, stream)] if F == 1 else [(G.iodf_create(model, B, device=local_rank, plan=G.IODF_PLAN_THROUGHPUT),
                                           torch.cuda.Stream(device=dev)) for _ in range(F)]
    one_lane = [(m, stream)]

    def timed_blocks(ln, blocks, steps):
        """`blocks` blocks of `steps` encodes dealt round-robin to the lanes `ln`; the events between blocks
        (on the main stream, which every lane's stream waits for before a block and is waited for after it)"""
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
        evs[0].record(stream)
        n = 0
        for b in range(blocks):
            for _, st in ln:
                if st is not stream:
                    st.wait_event(evs[b])
            for i in range(steps):
                mk, st = ln[n % len(ln)]
                G.iodf_forward(mk, xs[n % N_SETS], zs[n % N_SETS], ps[n % N_SETS], stream=st)
                n += 1
            for _, st in ln:
                if st is not stream:
                    e = torch.cuda.Event()
                    e.record(st)
                    stream.wait_event(e)
            evs[b + 1].record(stream)
        return evs

    for i in range(max(args.warmup, F)):
        mk, st = lanes[i % F]
        G.iodf_forward(mk, xs[i % N_SETS], zs[i % N_SETS], ps[i % N_SETS], stream=st)
    for i in range(args.warmup):
        G.iodf_forward(m, xs[i % N_SETS], zs[i % N_SETS], ps[i % N_SETS])
    torch.cuda.synchronize()
    for mk, _ in lanes + one_lane:
        G.iodf_check(mk)
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record(stream)
    for i in range(3):
        G.iodf_forward(m, xs[i % N_SETS], zs[i % N_SETS], ps[i % N_SETS])
    w1.record(stream)
    w1.synchronize()
    est_ms = max(w0.elapsed_time(w1) / 3.0, 1e-3)
    blocks = int(min(200, max(5, np.ceil(250.0 / (est_ms * args.steps)))))
    blocks = int(max_over_ranks([blocks], world, dev)[0])
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    evs = timed_blocks(lanes, blocks, args.steps)
    barrier()
    block_ms = sorted(evs[b].elapsed_time(evs[b + 1]) for b in range(blocks))
    total_ms = block_ms[len(block_ms) // 2]          # the median block of `steps` steps
    min_ms = block_ms[0]
    sampler.stop_flag = True
    sampler.join()
    for mk, _ in lanes:
        G.iodf_check(mk)
    # the same steps one after the other on one stream: the time of a step alone
    evs = timed_blocks(one_lane, 5, args.steps)
    barrier()
    one_ms = sorted(evs[b].elapsed_time(evs[b + 1]) for b in range(5))[2]
    for mk, _ in lanes:
        if mk is not m:
            G.iodf_destroy(mk)

    # ---- dominant kernel, timed alone per launch with events on the same stream --------------
    lvl = np.zeros(int(lay.n_levels))
    reps = min(50, max(5, args.steps))
    for i in range(reps):
        lvl += np.array(G.iodf_forward_timed(m, xs[i % N_SETS], zs[i % N_SETS], ps[i % N_SETS]))
    lvl /= reps
    top = int(np.argmax(lvl))
    lv = model["levels"][top]
    px = lv["h"] * lv["w"]
    top_macs = sum(px * ly["k"] ** 2 * ly["c_in"] * ly["c_out"] for cp in lv["couplings"] for ly in cp["layers"])
    if lv["prior"] is not None:
        ly = lv["prior"]["layer"]
        top_macs += px * 9 * ly["c_in"] * ly["c_out"]
    hbm, bf16, which = peaks()
    # the roofline's denominator: this GPU's int8 tensor pipe, measured by the library's MMA-only
    # kernel in this run; 2 x the bf16 figure (nominal dense int8 : bf16 = 2 : 1) is the cross-check
    peak_burst, peak_sustained = measure_int8_peak(G, m, stream, torch)
    peak_int8 = peak_burst                      # a step is far below a second: the burst figure applies
    achieved = 2.0 * top_macs * B / (lvl[top] * 1e-3) / 1e12
    traffic, traffic_note = stored_traffic("config%s_b%d_level%d" % (cfg, B, top))
    roofline = {"bound": "tensor", "kernel": "%s<encode> level %d" % (G.iodf_level_kernel_name(m, top), top),
                "achieved": achieved, "peak": peak_int8, "unit": "TOP/s (int8)", "frac": achieved / peak_int8,
                "traffic": traffic, "traffic_note": traffic_note,
                "peak_source": "tcgen05.mma kind::i8 128x256x32 MMA-only kernel, all SMs, measured in this run (burst: best ~10 ms launch)",
                "peak_sustained": peak_sustained,
                "peak_crosscheck": {"value": 2.0 * bf16, "what": "2 x %s burst bf16 %.1f TFLOP/s" % (which, bf16)},
                "level_ms": [float(v) for v in lvl],
                "whole_step_frac": (2.0 * macs * B / (total_ms / args.steps * 1e-3) / 1e12) / peak_int8}

    # ---- decode of the same workload, and batch-1 latency of both directions ------------------
    # zs hold valid latents of the encoded sets; the decoder must give the images back.
    xo = [torch.empty_like(xs[0]) for _ in range(N_SETS)]
    dec_steps = max(10, min(args.steps, 200))
    for i in range(max(3, min(args.warmup, 10))):
        G.iodf_inverse(m, zs[i % N_SETS], xo[i % N_SETS])
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record(stream)
    for i in range(dec_steps):
        G.iodf_inverse(m, zs[i % N_SETS], xo[i % N_SETS])
    d1.record(stream)
    barrier()
    dec_ms = d0.elapsed_time(d1)
    G.iodf_check(m)
    dec_ok = bool(all(torch.equal(xo[i], xs[i]) for i in range(min(N_SETS, args.steps + args.warmup))))

    def latency_b1(fn):
        ts = []
        for i in range(23):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(i % N_SETS)
            b.record(stream)
            b.synchronize()
            ts.append(a.elapsed_time(b))
        ts = sorted(ts[3:])
        return {"median_ms": ts[len(ts) // 2], "min_ms": ts[0]}
    lat = {"encode": latency_b1(lambda i: G.iodf_forward(m, xs[i][:1], zs[i][:1], ps[i][:1])),
           "decode": latency_b1(lambda i: G.iodf_inverse(m, zs[i][:1], xo[i][:1]))}
    G.iodf_check(m)

    # ---- level-stepped decode and patch-based encode of the same workload (single GPU) -----------
    extra = {}
    if world == 1:
        def timed(fn, n):
            for i in range(3):
                fn(i)
            t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            t0e.record(stream)
            for i in range(n):
                fn(i)
            t1e.record(stream)
            t1e.synchronize()
            return t0e.elapsed_time(t1e) / n
        L = int(lay.n_levels)
        has_prior = [lv["prior"] is not None for lv in model["levels"]]

        def stepped(i):
            k = i % N_SETS
            for lv in range(L - 1, -1, -1):
                if has_prior[lv]:
                    G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, zs[k], prior=ps[k])
                G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, zs[k], x_u8=xo[k])
        ms = timed(stepped, dec_steps)
        ok = bool(all(torch.equal(xo[i], xs[i]) for i in range(min(N_SETS, args.steps + args.warmup))))   # the sets that were encoded
        extra["decode_level_stepped"] = {"value": B / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
                                         "launches_per_step": L + sum(has_prior), "round_trip_exact": ok}
        # the batch as the patch grid of one image: patches_y x patches_x patches of the model's input size
        px_ = 1
        while px_ * px_ < B:
            px_ *= 2
        py_ = B // px_
        if px_ * py_ == B:
            hw = model["in_h"]
            imgs = [x.reshape(py_, px_, 3, hw, hw).permute(2, 0, 3, 1, 4).reshape(3, py_ * hw, px_ * hw).contiguous()
                    for x in xs]
            zp, pp = G.iodf_forward_patches(m, imgs[0])
            same = bool(torch.equal(zp, G.iodf_forward(m, xs[0])[0]))
            ms = timed(lambda i: G.iodf_forward_patches(m, imgs[i % N_SETS], zs[i % N_SETS], ps[i % N_SETS]),
                       dec_steps)
            extra["encode_patches"] = {"image": "3x%dx%d" % (py_ * hw, px_ * hw), "patches": B, "ms_per_image": ms,
                                       "value": 3.0 * py_ * hw * px_ * hw / (ms * 1e-3) / 1e6, "unit": "MB/s",
                                       "equals_batch_encode": same}
        # entropy coding of the latents (rANS, one thread per stream) and the whole compressor /
        # decompressor: flow + coder, latents and prior parameters never leave the GPU
        codec = S.logistic_codec()
        cd = G.iodf_codec_create(m, codec)
        wbuf = [torch.empty((B, cd.n_streams, cd.words_per_stream), dtype=torch.int16, device=dev) for _ in range(2)]
        cbuf = [torch.empty((B, cd.n_streams), dtype=torch.int32, device=dev) for _ in range(2)]
        G.iodf_forward(m, xs[0], zs[0], ps[0])
        enc_ms = timed(lambda i: G.iodf_rans_encode(cd, zs[0], ps[0], wbuf[i % 2], cbuf[i % 2]), dec_steps)
        blk_of = {int(cd.layout.block_level[q]): q for q in range(cd.n_blocks - 1)}

        def compress(i):
            k = i % N_SETS
            G.iodf_forward(m, xs[k], zs[k], ps[k])
            G.iodf_rans_encode(cd, zs[k], ps[k], wbuf[0], cbuf[0])

        def decompress(i):
            k = 0
            G.iodf_rans_decode_block(cd, cd.n_blocks - 1, wbuf[1], cbuf[1], ps[k], zs[k])
            for lv in range(L - 1, -1, -1):
                if lv in blk_of:
                    G.iodf_inverse_level(m, lv, G.IODF_LEVEL_PRIOR, zs[k], prior=ps[k])
                    G.iodf_rans_decode_block(cd, blk_of[lv], wbuf[1], cbuf[1], ps[k], zs[k])
                G.iodf_inverse_level(m, lv, G.IODF_LEVEL_COUPLINGS, zs[k], x_u8=xo[k])
        G.iodf_forward(m, xs[0], zs[0], ps[0])
        G.iodf_rans_encode(cd, zs[0], ps[0], wbuf[1], cbuf[1])
        coded_bytes = 2.0 * float(cbuf[1].to(torch.int64).sum().item())
        zs[0].fill_(0x7A7A7A7A)
        dms = timed(decompress, dec_steps)
        rt = bool(torch.equal(xo[0], xs[0]))
        cms = timed(compress, dec_steps)
        G.iodf_codec_check(cd)
        raw = float(B * m.d)
        # The same with four batches in flight, each with a model handle (throughput plan), a codec, a
        # stream and buffers of its own: one batch's block decodes run under the others' flow kernels.
        CL = 4
        cl = []
        for k in range(CL):
            mk = G.iodf_create(model, B, device=local_rank, plan=G.IODF_PLAN_THROUGHPUT)
            ck = G.iodf_codec_create(mk, codec)
            zk, pk_ = G.iodf_forward(mk, xs[k])
            wk, nk = G.iodf_rans_encode(ck, zk, pk_)
            cl.append(dict(m=mk, cd=ck, x=xs[k], w=wk, c=nk, st=torch.cuda.Stream(device=dev), xo=torch.empty_like(xs[k]),
                           z=torch.empty_like(zk), p=torch.empty_like(pk_), w2=torch.empty_like(wk), c2=torch.empty_like(nk)))
        torch.cuda.synchronize()

        def decompress_lane(l):
            G.iodf_rans_decode_block(l["cd"], cd.n_blocks - 1, l["w"], l["c"], l["p"], l["z"], stream=l["st"])
            for lv in range(L - 1, -1, -1):
                if lv in blk_of:
                    G.iodf_inverse_level(l["m"], lv, G.IODF_LEVEL_PRIOR, l["z"], prior=l["p"], stream=l["st"])
                    G.iodf_rans_decode_block(l["cd"], blk_of[lv], l["w"], l["c"], l["p"], l["z"], stream=l["st"])
                G.iodf_inverse_level(l["m"], lv, G.IODF_LEVEL_COUPLINGS, l["z"], x_u8=l["xo"], stream=l["st"])

        def compress_lane(l):
            G.iodf_forward(l["m"], l["x"], l["z"], l["p"], stream=l["st"])
            G.iodf_rans_encode(l["cd"], l["z"], l["p"], l["w2"], l["c2"], stream=l["st"])

        def timed_lanes(fn, n):
            def run(n):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for l in cl:
                    l["st"].wait_event(e0)
                for i in range(n):
                    fn(cl[i % CL])
                for l in cl:
                    e = torch.cuda.Event()
                    e.record(l["st"])
                    stream.wait_event(e)
                e1.record(stream)
                e1.synchronize()
                return e0.elapsed_time(e1) / n
            run(2 * CL)
            return run(n)
        for l in cl:
            l["z"].fill_(0x7A7A7A7A)
        dms_f = timed_lanes(decompress_lane, dec_steps)
        rt_f = all(bool(torch.equal(l["xo"], l["x"])) for l in cl)
        cms_f = timed_lanes(compress_lane, dec_steps)
        rt_f = rt_f and all(bool(torch.equal(l["c2"], l["c"])) for l in cl)
        for l in cl:
            G.iodf_codec_check(l["cd"])
            G.iodf_check(l["m"])
            G.iodf_destroy(l["m"])
        # the oracle's coder on a few images of the same latents, for the CPU figure beside it
        import oracle as O
        nz = min(B, 8)
        zc, pc = zs[0][:nz].cpu().numpy(), ps[0][:nz].cpu().numpy()
        G.iodf_forward(m, xs[0], zs[0], ps[0])
        zc, pc = zs[0][:nz].cpu().numpy(), ps[0][:nz].cpu().numpy()
        t0 = time.perf_counter()
        O.rans_encode(codec, model, zc, pc)
        cpu_s = time.perf_counter() - t0
        # host images -> host byte stream -> host images, pinned buffers, one synchronise per call
        hxi = torch.from_numpy(S.config_images(cfg, batch=B)).pin_memory()
        hout = torch.empty(G.iodf_rans_packed_capacity(cd, B), dtype=torch.uint8).pin_memory()
        hback = torch.empty_like(hxi).pin_memory()
        nb = 0
        for _ in range(3):
            _, nb = G.iodf_compress_host(m, cd, hxi, out_host=hout)
        n_h = max(10, min(args.steps, 50))
        t0 = time.perf_counter()
        for _ in range(n_h):
            G.iodf_compress_host(m, cd, hxi, out_host=hout)
        ch_s = (time.perf_counter() - t0) / n_h
        for _ in range(3):
            G.iodf_decompress_host(m, cd, hout, nb, B, x_u8_host=hback)
        stream.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_h):
            G.iodf_decompress_host(m, cd, hout, nb, B, x_u8_host=hback)
            stream.synchronize()
        dh_s = (time.perf_counter() - t0) / n_h
        G.iodf_codec_check(cd)
        host_rt = bool(torch.equal(hback, hxi))
        extra["entropy_coding"] = {
            "compress_host_MB_per_s": raw / ch_s / 1e6, "decompress_host_MB_per_s": raw / dh_s / 1e6,
            "compressed_bytes_per_batch": nb, "host_round_trip_exact": host_rt,
            "rans_encode_ms": enc_ms, "rans_encode_msym_per_s": B * m.d / (enc_ms * 1e-3) / 1e6,
            "streams": B * cd.n_streams, "bits_per_dim": 8.0 * coded_bytes / raw,
            "note": "random (untrained) weights: the bit rate says nothing about the model, only that the coder is exact",
            "batches_in_flight": CL,
            "compress_ms": cms_f, "compress_MB_per_s": raw / (cms_f * 1e-3) / 1e6,
            "decompress_ms": dms_f, "decompress_MB_per_s": raw / (dms_f * 1e-3) / 1e6, "round_trip_exact": rt and rt_f,
            "one_batch_at_a_time": {"compress_ms": cms, "compress_MB_per_s": raw / (cms * 1e-3) / 1e6,
                                    "decompress_ms": dms, "decompress_MB_per_s": raw / (dms * 1e-3) / 1e6},
            "cpu_oracle_rans_msym_per_s": nz * m.d / cpu_s / 1e6}
        G.iodf_check(m)

    # ---- end to end through the host-buffer entry point --------------------------------------
    hx = [torch.from_numpy(S.config_images(cfg, batch=B, seed_offset=rank_seed_offset(rank, i))).pin_memory() for i in range(2)]
    hz = [torch.empty((B, m.d), dtype=torch.int32).pin_memory() for _ in range(2)]
    hp = [torch.empty((B, 2, m.d_fact), dtype=torch.int32).pin_memory() for _ in range(2)]
    e2e_steps = max(10, min(args.steps, 100))
    for i in range(3):
        G.iodf_forward_host(m, hx[i % 2], hz[i % 2], hp[i % 2])
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        G.iodf_forward_host(m, hx[i % 2], hz[i % 2], hp[i % 2])
        stream.synchronize()      # the result is read on the host every step
    barrier()
    e2e_s = time.perf_counter() - t0
    G.iodf_check(m)
    # The same with four calls in flight, each on a stream, a model handle and a set of pinned host
    # buffers of its own, so that a step's device-to-host copy runs under the next steps' uploads and
    # kernels. Every step still uploads its inputs from pinned host memory, and its result is on the
    # host before its buffers are reused.
    E = 4
    hx += [torch.from_numpy(S.config_images(cfg, batch=B, seed_offset=rank_seed_offset(rank, i))).pin_memory() for i in range(2, E)]
    hz += [torch.empty((B, m.d), dtype=torch.int32).pin_memory() for _ in range(2, E)]
    hp += [torch.empty((B, 2, m.d_fact), dtype=torch.int32).pin_memory() for _ in range(2, E)]
    hlanes = [(G.iodf_create(model, B, device=local_rank, plan=G.IODF_PLAN_THROUGHPUT), torch.cuda.Stream(device=dev))
              for _ in range(E)]
    for i in range(2 * E):
        G.iodf_forward_host(hlanes[i % E][0], hx[i % E], hz[i % E], hp[i % E], stream=hlanes[i % E][1])
    for _, st in hlanes:
        st.synchronize()
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        mk, st = hlanes[i % E]
        st.synchronize()          # step i - E of this lane is complete: its result has been read
        G.iodf_forward_host(mk, hx[i % E], hz[i % E], hp[i % E], stream=st)
    for _, st in hlanes:
        st.synchronize()
    barrier()
    e2e2_s = time.perf_counter() - t0
    for mk, _ in hlanes:
        G.iodf_check(mk)
    e2e_same = not bool(torch.equal(hz[0], hz[1]))      # the lanes had different inputs: different latents
    for mk, _ in hlanes:
        G.iodf_destroy(mk)

    total_ms, min_ms, one_ms, e2e_s, e2e2_s, dec_ms = max_over_ranks([total_ms, min_ms, one_ms, e2e_s, e2e2_s, dec_ms], world, dev)

    if rank == 0:
        cores = os.cpu_count() or 1
        out = {
            "metric": METRIC, "value": job_throughput(B, world, args.steps, total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "ms_per_step_min": min_ms / args.steps, "timed_blocks": blocks,
            "timing": "median over %d blocks of %d steps, each block between CUDA events; %d steps in flight (a stream "
                      "and a model handle, made with the throughput plan, each)" % (blocks, args.steps, F),
            "steps_in_flight": F,
            "one_step_at_a_time": {"ms_per_step": one_ms / args.steps, "value": job_throughput(B, world, args.steps, one_ms * 1e-3)},
            "ms_per_sample": total_ms / args.steps / B,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": dict(workload(args), steps_in_flight=F), "clocks": sampler.summary(), "roofline": roofline,
            "e2e": {"value": job_throughput(B, world, e2e_steps, e2e2_s), "unit": UNIT, "h2d_bytes_per_step": B * m.d,
                    "d2h_bytes_per_step": B * m.d * 4 + B * 2 * m.d_fact * 4, "steps": e2e_steps,
                    "how": "iodf_forward_host, pinned host buffers, four calls in flight (a model handle and a stream each)",
                    "one_call_at_a_time": job_throughput(B, world, e2e_steps, e2e_s), "lanes_distinct": e2e_same},
            "gpu_launches": G.iodf_launches_per_call(m) * args.steps,
            "gpu_launches_all_blocks": G.iodf_launches_per_call(m) * args.steps * blocks,
            "gops_per_image": 2.0 * macs / 1e9,
            "decode": {"metric": "flow_decode_images_per_sec", "value": job_throughput(B, world, dec_steps, dec_ms * 1e-3),
                       "unit": UNIT, "ms_per_step": dec_ms / dec_steps, "steps": dec_steps,
                       "round_trip_exact": dec_ok},
            "latency_batch1": lat,
        }
        out.update(extra)
        if cfg == "R32":
            # the paper's own latency for this architecture, for context only: another GPU, a trained
            # model, floating-point requantisation, the first conv of every coupling in FP32
            out["paper_context"] = {"ms_per_sample": 0.27, "batch": 64, "hardware": "Tesla T4, TensorRT 8.2",
                                    "source": "Table 4, IODF on ImageNet32"}
        if world == 1:
            r, n, dt = oracle_rate(model, cfg, B, cores, seconds=10.0)
            out["cpu_baseline"] = {"value": r, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": "%d images of the same workload, oracle forward, %.1f s" % (n, dt)}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
