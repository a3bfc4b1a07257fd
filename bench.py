#!/usr/bin/env python
"""Benchmark of the layer-parallel training step on B200 (one process per GPU).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload wrn28_10] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic batch: AuxNet forward chain, all K
modules' forward + local loss + backward (concurrently, on K streams), parameter / multiplier
update.  The step is recorded once into a CUDA graph and replayed.  `value` is images/s with the
inputs resident in HBM; `e2e` is the same step driven from pinned host buffers (images and labels
copied in, the K losses copied out, every step).  With N > 1 the ranks are independent replicas
(the path does not shard: no collective), and `value` is the sum over ranks.

`--impl reference` times the CPU oracle (oracle/lp_oracle.py, as it stands) on a bounded sample of
the same workload on the host cores.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "images/sec per layer-parallel step"
UNIT = "images/s"


def recorded_traffic(workload):
    """DRAM bytes per launch of the dominant kernel as the last profiler capture recorded them: the
    `traffic_bytes_per_launch:` line of profiles/conv_tc_kernel_traffic.md (with the workload, kernel and
    source revision it was taken at).  None when there is no such record for this workload."""
    path = os.path.join(ROOT, "profiles", "conv_tc_kernel_traffic.md")
    if not os.path.exists(path):
        return None, None
    rec = {}
    for line in open(path):
        if ":" in line and line.split(":", 1)[0].strip() in ("traffic_bytes_per_launch", "workload", "kernel", "revision"):
            k, v = line.split(":", 1)
            rec[k.strip()] = v.strip()
    if rec.get("workload") != workload or "traffic_bytes_per_launch" not in rec:
        return None, None
    return float(rec["traffic_bytes_per_launch"]), "%s at revision %s (profiles/conv_tc_kernel_traffic.md)" % (
        rec.get("kernel", "?"), rec.get("revision", "?"))


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wrn28_10")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (0 = the workload's own)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-serial", action="store_true")
    ap.add_argument("--conv-impl", type=int, default=0)
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="the timed region of --steps steps is repeated until this much time has been measured; the "
                         "median repeat is reported")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------
# workload FLOP accounting (true sizes, multiply-add = 2 FLOPs, backward = 2 x forward)
# ---------------------------------------------------------------------------------------------
def conv_flops_forward(cfg):
    """Forward conv FLOPs per step: main network (stem + blocks) and AuxNet, from the oracle-free
    shape walk below (this is bookkeeping for the report, not part of the path)."""
    def out(h, r, s, p):
        return (h + 2 * p - r) // s + 1
    n = cfg["N"]
    h, w = cfg["H"], cfg["W"]
    fl = 0.0
    if cfg["stem_kind"] == "conv3x3":
        fl += 2.0 * n * h * w * cfg["stem_channels"] * 9 * cfg["C_in"]
    else:
        h, w = out(h, 7, 2, 3), out(w, 7, 2, 3)
        fl += 2.0 * n * h * w * cfg["stem_channels"] * 49 * cfg["C_in"]
        h, w = out(h, 3, 2, 1), out(w, 3, 2, 1)
    c = cfg["stem_channels"]
    shapes = []
    for ch, nb, st in zip(cfg["stage_channels"], cfg["stage_blocks"], cfg["stage_stride"]):
        for b in range(nb):
            s = st if b == 0 else 1
            shapes.append((h, w, c))
            ho, wo = out(h, 3, s, 1), out(w, 3, s, 1)
            fl += 2.0 * n * ho * wo * ch * 9 * c + 2.0 * n * ho * wo * ch * 9 * ch
            if s != 1 or c != ch:
                fl += 2.0 * n * ho * wo * ch * c
            h, w, c = ho, wo, ch
    # AuxNet
    aux = 0.0
    ends = cfg["module_block_end"]
    bshape = [(cfg["H"], cfg["W"], cfg["C_in"])] + [shapes[e] for e in ends[:-1]]
    for k in range(len(ends) - 1):
        (hi, wi, ci), (ho, wo, co) = bshape[k], bshape[k + 1]
        total = hi // ho
        if cfg["aux_convs"] == 1:
            aux += 2.0 * n * ho * wo * co * 9 * ci
        else:
            hid = co // cfg["aux_width_div"]
            s1 = 2 if total >= 2 else 1
            hm, wm = out(hi, 3, s1, 1), out(wi, 3, s1, 1)
            aux += 2.0 * n * hm * wm * hid * 9 * ci + 2.0 * n * ho * wo * co * 9 * hid
    return fl, aux


# ---------------------------------------------------------------------------------------------
# clocks sampling during the timed region
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (bounded sample)
# ---------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle_step(cfg_name, sample_batch, repeats=1):
    """One layer-parallel step of the oracle (AuxNet chain, K module forward+backward, updates) on
    `sample_batch` images of the workload; returns (images/s, seconds per step)."""
    from oracle import lp_oracle as O
    from workloads import gen, scaled
    cfg = scaled(cfg_name, N=sample_batch)
    net = O.Net(cfg)
    mods = [gen.make_params(net.param_layout(k), 0, "module%d" % k) for k in range(net.K)]
    auxs = [gen.make_params(net.param_layout(O.LP_AUX(k)), 0, "aux%d" % k) for k in range(net.K - 1)]
    images, labels = gen.make_images(cfg), gen.make_labels(cfg)
    kappas = None
    if cfg["loss"] == "al":
        kappas = [np.zeros(net.boundary[k + 1]) for k in range(net.K - 1)]
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.layer_parallel_step(net, mods, auxs, images, labels, kappas, cfg["rho"], 1e-4)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return sample_batch / best, best


def oracle_sample_batch(cfg):
    # about 10-30 s of CPU work: the oracle sustains roughly 50-100 GFLOP/s of fp64 matmul
    fwd, aux = conv_flops_forward(cfg)
    per_image = (3 * fwd + aux) / cfg["N"]
    target = 1.2e12
    return int(max(1, min(cfg["N"], target // per_image)))


def run_reference(args):
    from workloads import get_config
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_config(args.workload)
    sb = oracle_sample_batch(cfg)
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    for _ in range(warm):
        time_oracle_step(args.workload, sb)
    times = [time_oracle_step(args.workload, sb)[1] for _ in range(steps)]
    dt = float(np.mean(times))
    val = sb / dt
    line = {"metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warm,
            "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": args.workload, "sample_batch": sb, "full_batch": cfg["N"]},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                             "sample": "one full layer-parallel step on %d of %d images" % (sb, cfg["N"])},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# aggregation over replicas (the only cross-rank step: no data-path collective)
# ---------------------------------------------------------------------------------------------
def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum of a list of per-rank scalars over all ranks (identity without dist)."""
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_images_per_s(batch_per_rank, steps, world, ms_max_over_ranks):
    """Every rank processes `batch_per_rank` images per step; the job is as slow as its slowest rank."""
    return batch_per_rank * steps * world / (ms_max_over_ranks * 1e-3)


# ---------------------------------------------------------------------------------------------
# GPU benchmark
# ---------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import paper_2112_05387_b200 as lp
    from workloads import gen, get_config, scaled

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    cfg = scaled(args.workload, N=args.batch) if args.batch else get_config(args.workload)
    K = cfg["K"]
    desc = lp.desc_from_config(cfg, args.conv_impl)
    h = lp.lp_create(desc, device=str(dev))
    tdt = torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16
    for k in range(K):
        lp.lp_set_params(h, k, gen.make_params(lp.lp_param_layout(desc, k), 0, "module%d" % k, dtype=cfg["dtype"]))
    for k in range(K - 1):
        lp.lp_set_params(h, lp.LP_AUX(k), gen.make_params(lp.lp_param_layout(desc, lp.LP_AUX(k)), 0, "aux%d" % k,
                                                         dtype=cfg["dtype"]))
    images_host = torch.from_numpy(gen.make_images(cfg)).to(tdt).pin_memory()
    labels_host = torch.from_numpy(gen.make_labels(cfg)).pin_memory()
    d_images = images_host.to(dev)
    d_labels = labels_host.to(dev)
    shapes = [lp.lp_boundary_shape_desc(desc, k) for k in range(K)]
    d_x = [d_images] + [torch.zeros(shapes[k], dtype=tdt, device=dev) for k in range(1, K)]
    use_kappa = cfg["loss"] == "al"
    d_kappa = [torch.zeros(shapes[k + 1], dtype=tdt, device=dev) for k in range(K - 1)] if use_kappa else None
    d_dx = [None] + [torch.zeros_like(d_x[k]) for k in range(1, K)]
    d_loss = torch.zeros(K, 2, dtype=torch.float32, device=dev)
    loss_host = torch.zeros(K, 2, dtype=torch.float32).pin_memory()
    lr = 1e-9  # the penalty is a sum over the boundary tensor: a small rate keeps replayed steps finite
    kstep = cfg["rho"]
    stream = torch.cuda.Stream(device=dev)
    sp = stream.cuda_stream

    def step_direct():
        # the whole step in one call: AuxNet on its own stream, every module starting, taking its
        # loss and updating as soon as its own inputs exist
        lp.lp_layer_parallel_step(h, d_images, d_x[1:], d_labels, d_kappa, cfg["rho"], d_loss, d_dx, lr, 0.0, 0.0,
                                  kstep, sp)

    def step_three_calls():
        lp.lp_auxnet_forward(h, d_images, d_x[1:], sp)
        lp.lp_modules_fwd_bwd_all(h, d_x, d_labels, d_kappa, cfg["rho"], d_loss, d_dx, sp)
        lp.lp_step(h, lr, 0.0, 0.0, kstep, d_kappa, sp)

    def serial_direct():
        lp.lp_serial_fwd_bwd(h, d_images, d_labels, d_loss[K - 1], sp)
        lp.lp_step(h, lr, 0.0, 0.0, 0.0, None, sp)

    with torch.cuda.stream(stream):
        step_direct()                       # first use sets kernel attributes, outside any capture
        st = lp.lp_last_device_status(h, sp)
        if st != 0:
            raise RuntimeError("device status %d after the first step" % st)
        lp.lp_launch_count(h, reset=True)
        step_direct()
        launches_per_step = lp.lp_launch_count(h, reset=True)
        gid = None
        if not args.no_graph:
            lp.lp_graph_begin(h, sp)
            step_direct()
            gid = lp.lp_graph_end(h, sp)

        def step():
            if gid is None:
                step_direct()
            else:
                lp.lp_graph_launch(h, gid, sp)

        def barrier():
            torch.cuda.synchronize(dev)
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize(dev)

        for _ in range(max(args.warmup, 3)):
            step()
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        # The timed region (exactly `steps` steps between two events, a barrier and a synchronize on both
        # sides) is repeated until at least --min-seconds have been measured, so that the part reaches its
        # steady clock and power; the median repeat is the reported one.
        reps_ms = []
        while True:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                step()
            e1.record(stream)
            barrier()
            reps_ms.append(e0.elapsed_time(e1))
            if sum(reps_ms) >= args.min_seconds * 1e3 or len(reps_ms) >= 1000:
                break
        ms = float(np.median(reps_ms))
        clocks = sampler.stop()
        st = lp.lp_last_device_status(h, sp)
        if st != 0:
            raise RuntimeError("device status %d in the timed region" % st)

        # end to end: pinned host inputs in, losses out, every step
        for _ in range(2):
            d_images.copy_(images_host, non_blocking=True)
            d_labels.copy_(labels_host, non_blocking=True)
            step()
            loss_host.copy_(d_loss, non_blocking=True)
        barrier()
        # same scheme as above: the region of `steps` steps is repeated until half of --min-seconds has been
        # measured, and the median repeat is reported
        e2e_reps = []
        while True:
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            for _ in range(args.steps):
                d_images.copy_(images_host, non_blocking=True)
                d_labels.copy_(labels_host, non_blocking=True)
                step()
                loss_host.copy_(d_loss, non_blocking=True)
                stream.synchronize()             # the caller reads the losses before the next step
            f1.record(stream)
            barrier()
            e2e_reps.append(f0.elapsed_time(f1))
            if sum(e2e_reps) >= 0.5 * args.min_seconds * 1e3 or len(e2e_reps) >= 1000:
                break
        ms_e2e = float(np.median(e2e_reps))
        losses = loss_host.clone().numpy()

        # per-kernel timing of the tensor-core convolutions: modules one after another on one
        # stream (so that a kernel's events do not include waiting for another module's kernels)
        lp.lp_conv_profile(h, True, read=False)
        prof_steps = 2
        for _ in range(prof_steps):
            lp.lp_auxnet_forward(h, d_images, d_x[1:], sp)
            for k in range(K):
                last = k == K - 1
                lp.lp_module_fwd_bwd(h, k, d_x[k], d_labels if last else d_x[k + 1],
                                     None if (last or not use_kappa) else d_kappa[k], cfg["rho"], d_loss[k],
                                     d_dx[k], sp)
        conv_ms, conv_flops, conv_launches = lp.lp_conv_profile(h, False, read=True)
        barrier()

        # what an event pair costs around a launch that does nothing: the part of every per-launch time above that
        # is not the kernel's own work (the stream is kept busy before each pair so that the host is ahead)
        busy = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
        tiny = torch.zeros(1, dtype=torch.float32, device=dev)
        floors = []
        for _ in range(24):
            busy.zero_()
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            tiny.zero_()
            f1.record(stream)
            stream.synchronize()
            floors.append(f0.elapsed_time(f1))
        event_pair_floor_ms = float(np.median(floors[4:]))
        del busy

        # per-operation time line of the same serial pass: achieved GB/s of the HBM-bound kernels
        # (algorithmic bytes of the operation / its CUDA-event time)
        lp.lp_timeline(h, True, read=False)
        tl_steps = 3
        for _ in range(tl_steps):
            lp.lp_auxnet_forward(h, d_images, d_x[1:], sp)
            for k in range(K):
                last = k == K - 1
                lp.lp_module_fwd_bwd(h, k, d_x[k], d_labels if last else d_x[k + 1],
                                     None if (last or not use_kappa) else d_kappa[k], cfg["rho"], d_loss[k],
                                     d_dx[k], sp)
            lp.lp_step(h, lr, 0.0, 0.0, kstep, d_kappa, sp)
        tl_recs = lp.lp_timeline(h, False, read=True, max_records=20000)
        barrier()

        distill = None
        if not args.no_serial and world == 1 and K > 1:
            d_dloss = torch.zeros(K - 1, dtype=torch.float32, device=dev)

            def step_with_distill():
                step_direct()
                lp.lp_auxnet_distill(h, d_images, d_x[1:], d_dx, 1e-9, 1e-9, None, d_dloss, sp)
            step_with_distill()
            dgid = None
            if not args.no_graph:
                lp.lp_graph_begin(h, sp)
                step_with_distill()
                dgid = lp.lp_graph_end(h, sp)
            for _ in range(3):
                lp.lp_graph_launch(h, dgid, sp) if dgid is not None else step_with_distill()
            barrier()
            d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_d = max(3, args.steps // 3)
            d0.record(stream)
            for _ in range(n_d):
                lp.lp_graph_launch(h, dgid, sp) if dgid is not None else step_with_distill()
            d1.record(stream)
            barrier()
            distill = {"value": cfg["N"] * n_d / (d0.elapsed_time(d1) * 1e-3), "unit": UNIT,
                       "what": "the step followed by lp_auxnet_distill (auxiliary-variable correction + one AuxNet "
                               "distillation step per boundary): all of Algorithm 1"}

        three = None
        if not args.no_serial and world == 1:
            step_three_calls()
            tgid = None
            if not args.no_graph:
                lp.lp_graph_begin(h, sp)
                step_three_calls()
                tgid = lp.lp_graph_end(h, sp)
            for _ in range(3):
                lp.lp_graph_launch(h, tgid, sp) if tgid is not None else step_three_calls()
            barrier()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_t = max(3, args.steps // 3)
            t0.record(stream)
            for _ in range(n_t):
                lp.lp_graph_launch(h, tgid, sp) if tgid is not None else step_three_calls()
            t1.record(stream)
            barrier()
            three = {"value": cfg["N"] * n_t / (t0.elapsed_time(t1) * 1e-3), "unit": UNIT,
                     "what": "lp_auxnet_forward + lp_modules_fwd_bwd_all + lp_step as three calls (AuxNet and update not overlapped)"}

        serial = None
        if not args.no_serial and world == 1:
            serial_direct()
            sgid = None
            if not args.no_graph:
                lp.lp_graph_begin(h, sp)
                serial_direct()
                sgid = lp.lp_graph_end(h, sp)
            for _ in range(3):
                lp.lp_graph_launch(h, sgid, sp) if sgid is not None else serial_direct()
            barrier()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_ser = max(3, args.steps // 3)
            g0.record(stream)
            for _ in range(n_ser):
                lp.lp_graph_launch(h, sgid, sp) if sgid is not None else serial_direct()
            g1.record(stream)
            barrier()
            serial = {"value": cfg["N"] * n_ser / (g0.elapsed_time(g1) * 1e-3), "unit": UNIT,
                      "what": "layer-serial forward + back-propagation + update with the same kernels (no AuxNet)"}

        # the same step with recursive AuxNets (Section 4.3): every x_k generated from the images by a
        # stack of its own on module k's stream, no serial AuxNet chain
        recursive = None
        if not args.no_serial and world == 1 and K > 2:
            rdesc = lp.desc_from_config(cfg, args.conv_impl, aux_recursive=True)
            hr = lp.lp_create(rdesc, device=str(dev))
            for k in range(K):
                lp.lp_set_params(hr, k, gen.make_params(lp.lp_param_layout(rdesc, k), 0, "module%d" % k, dtype=cfg["dtype"]))
            for k in range(1, K):
                for j in range(k):
                    w = lp.LP_REAUX(k, j)
                    lp.lp_set_params(hr, w, gen.make_params(lp.lp_param_layout(rdesc, w), 0, "reaux%d/%d" % (k, j),
                                                            dtype=cfg["dtype"]))

            def step_recursive():
                lp.lp_layer_parallel_step(hr, d_images, d_x[1:], d_labels, d_kappa, cfg["rho"], d_loss, d_dx, lr, 0.0,
                                          0.0, kstep, sp)
            step_recursive()
            rgid = None
            if not args.no_graph:
                lp.lp_graph_begin(hr, sp)
                step_recursive()
                rgid = lp.lp_graph_end(hr, sp)
            for _ in range(3):
                lp.lp_graph_launch(hr, rgid, sp) if rgid is not None else step_recursive()
            barrier()
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_r = max(3, args.steps // 3)
            r0.record(stream)
            for _ in range(n_r):
                lp.lp_graph_launch(hr, rgid, sp) if rgid is not None else step_recursive()
            r1.record(stream)
            barrier()
            if lp.lp_last_device_status(hr, sp) != 0:
                raise RuntimeError("device status in the recursive-AuxNet step")
            recursive = {"value": cfg["N"] * n_r / (r0.elapsed_time(r1) * 1e-3), "unit": UNIT,
                         "what": "the step with recursive AuxNets (one independent stack per boundary, K(K-1)/2 units)"}
            lp.lp_destroy(hr)

    # max over ranks
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dist, dev)
    reps_ms = [ms] if world > 1 else reps_ms
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = whole_job_images_per_s(cfg["N"], args.steps, world, ms)
    e2e_value = whole_job_images_per_s(cfg["N"], args.steps, world, ms_e2e)
    fwd, aux = conv_flops_forward(cfg)
    step_conv_flops = 3 * fwd + aux
    peaks = {}
    ppath = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak_src = "fallback"
    if os.path.exists(ppath):
        peaks = json.load(open(ppath))
        peak_src = "measured"
    peak_tf = float(peaks.get("bf16_tflops_sustained", 1400.0))
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    hbm_names = {"bn_apply": "bn_apply_kernel", "bn_bwd": "bn_bwd_reduce_kernel + bn_bwd_apply_kernel",
                 "bn_stats": "bn_stats_kernel", "out_loss": "module_out_loss_kernel",
                 "update": "sgd_pack_tiled64_kernel + sgd_ranges_kernel + kappa_update_kernel"}
    roofline_hbm = []
    for op, kernel in hbm_names.items():
        rs = [r for r in tl_recs if r["op"] == op and r["bytes"] > 0]
        if not rs:
            continue
        t_ms = sum(r["end_ms"] - r["start_ms"] for r in rs)
        nbytes = sum(r["bytes"] for r in rs)
        gbs = nbytes / (t_ms * 1e-3) / 1e9 if t_ms > 0 else 0.0
        roofline_hbm.append({"op": op, "kernel": kernel, "bound": "hbm", "launch_groups_timed": len(rs),
                             "ms_per_step": t_ms / tl_steps, "algorithmic_gb_per_step": nbytes / tl_steps / 1e9,
                             "achieved": gbs, "peak": peak_gbs, "unit": "GB/s", "frac": gbs / peak_gbs})
    traffic, traffic_src = recorded_traffic(args.workload if not args.batch else "")
    achieved_tf = conv_flops / (conv_ms * 1e-3) / 1e12 if conv_ms > 0 else 0.0
    roofline = {"bound": "tensor", "kernel": "conv_tc_kernel + wgrad_tc_kernel (all tensor-core convolutions)",
                "achieved": achieved_tf, "peak": peak_tf, "peak_source": peak_src + " (sustained bf16 GEMM)",
                "unit": "TFLOP/s", "frac": achieved_tf / peak_tf if peak_tf else None,
                "frac_of_nominal_2250": achieved_tf / 2250.0,
                "launches_timed": int(conv_launches), "avg_launch_ms": conv_ms / max(conv_launches, 1),
                "flops_per_launch_avg": conv_flops / max(conv_launches, 1),
                "traffic": traffic,
                "traffic_note": ("DRAM bytes read + written per launch, " + traffic_src) if traffic_src else
                                "no profiler record for this workload at the present kernels",
                "timing": "CUDA events around every tensor-core conv launch, modules run back to back on one stream",
                "event_pair_floor_ms": event_pair_floor_ms,
                "event_pair_floor_note": "a one-element fill between two CUDA events on the busy stream: this much of "
                                         "avg_launch_ms is launch and event latency, which a graph replay does not pay"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg["dtype"] == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": args.workload, "global_batch": cfg["N"] * world, "K": K, "loss": cfg["loss"],
                       "rho": cfg["rho"], "parallelism": "replicas only (no collective)" if world > 1 else "1 GPU",
                       "cuda_graph": gid is not None, "l2": "working set of a step (GBs) is far larger than L2",
                       "conv_flops_per_step": step_conv_flops},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": int(images_host.numel() * images_host.element_size() + labels_host.numel() * 4),
                    "d2h_bytes_per_step": int(loss_host.numel() * 4)},
            "gpu_launches": int(launches_per_step * args.steps),
            "launches_per_step": int(launches_per_step),
            "step_conv_tflops": step_conv_flops / (ms / args.steps * 1e-3) / 1e12,
            "timing": {"repeats": len(reps_ms), "seconds_timed": sum(reps_ms) * 1e-3, "reported": "median repeat",
                       "ms_per_step_min": min(reps_ms) / args.steps, "ms_per_step_max": max(reps_ms) / args.steps,
                       "ms_per_step_first": reps_ms[0] / args.steps,
                       "ms_per_step_x_sm_mhz": (ms / args.steps) * clocks["sm_mhz"] if clocks.get("sm_mhz") else None},
            "roofline": roofline,
            "roofline_hbm": roofline_hbm,
            "losses": [float(v) for v in losses[:, 0]]}
    if serial:
        line["layer_serial"] = serial
    if three:
        line["three_calls"] = three
    if distill:
        line["with_distillation"] = distill
    if recursive:
        line["recursive_auxnets"] = recursive
    if not args.no_cpu_baseline and world == 1:
        sb = oracle_sample_batch(cfg)
        val, dt = time_oracle_step(args.workload, sb)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": "one full layer-parallel step on %d of %d images (%.1f s)" % (sb, cfg["N"], dt)}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        import __graft_entry__ as g
        g.build()
        run_ours(args)


if __name__ == "__main__":
    main()
