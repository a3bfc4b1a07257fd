"""Speed-up accounting of the layer-parallel step on one GPU (Section 4.3 of the paper).

  python -m paper_2112_05387_b200.speedup_accounting --workload wrn28_10 --K 1 2 3 4 6 [--batch N]

For every K the network is split into K modules of equal block count and three things are measured:

* the phase times of the paper's cost table, each the sum of the CUDA-event durations of that
  phase's operations with the modules run one after another on one stream (so that nothing
  overlaps): T_f and T_b (forward / backward of all modules), t_psi (the interior local losses),
  t_f^lambda (AuxNet chain) and t_b^lambda (auxiliary-variable correction + AuxNet distillation);
* the step times: layer-serial back-propagation (K = 1 form of the same network, same kernels),
  the layer-parallel step, and the layer-parallel step followed by the distillation, all replayed
  as CUDA graphs;
* from these, the paper's speed-up ratio with T_d = 0 (inputs resident on the device),
      rho_model(K) = 1 / ( 1/K + (t_psi + t_f^lambda + t_b^lambda) / (T_f + T_b) ),
  which is what K devices would give, next to the ratio actually measured on ONE device, where the
  K modules share the GPU: serial step time / parallel step time.

One JSON line per K.  Inputs are the seeded synthetic batches of the workload.
"""
import argparse
import json


def _setup(lp, torch, gen, cfg, dev):
    K = cfg["K"]
    desc = lp.desc_from_config(cfg, 0)
    h = lp.lp_create(desc, device=str(dev))
    tdt = torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16
    for k in range(K):
        lp.lp_set_params(h, k, gen.make_params(lp.lp_param_layout(desc, k), 0, "module%d" % k, dtype=cfg["dtype"]))
    for k in range(K - 1):
        lp.lp_set_params(h, lp.LP_AUX(k), gen.make_params(lp.lp_param_layout(desc, lp.LP_AUX(k)), 0, "aux%d" % k,
                                                         dtype=cfg["dtype"]))
    s = {"h": h, "K": K, "cfg": cfg}
    s["images"] = torch.from_numpy(gen.make_images(cfg)).to(tdt).to(dev)
    s["labels"] = torch.from_numpy(gen.make_labels(cfg)).to(dev)
    shapes = [lp.lp_boundary_shape_desc(desc, k) for k in range(K)]
    s["x"] = [s["images"]] + [torch.zeros(shapes[k], dtype=tdt, device=dev) for k in range(1, K)]
    s["dx"] = [None] + [torch.zeros_like(s["x"][k]) for k in range(1, K)]
    s["kappa"] = ([torch.zeros(shapes[k + 1], dtype=tdt, device=dev) for k in range(K - 1)]
                  if cfg["loss"] == "al" else None)
    s["loss"] = torch.zeros(K, 2, dtype=torch.float32, device=dev)
    s["dloss"] = torch.zeros(max(K - 1, 1), dtype=torch.float32, device=dev)
    return s


def _time_graph(lp, torch, s, fn, stream, reps):
    h, sp = s["h"], stream.cuda_stream
    fn()
    lp.lp_graph_begin(h, sp)
    fn()
    gid = lp.lp_graph_end(h, sp)
    for _ in range(3):
        lp.lp_graph_launch(h, gid, sp)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        lp.lp_graph_launch(h, gid, sp)
    e1.record(stream)
    torch.cuda.synchronize()
    if lp.lp_last_device_status(h, sp) != 0:
        raise RuntimeError("device status")
    return e0.elapsed_time(e1) / reps


def measure(workload, K, batch=0, reps=30):
    import torch
    import paper_2112_05387_b200 as lp
    from workloads import gen, with_modules
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    kw = {"N": batch} if batch else {}
    cfg = with_modules(workload, K, **kw)
    s = _setup(lp, torch, gen, cfg, dev)
    h, rho, lr = s["h"], cfg["rho"], 1e-9
    stream = torch.cuda.Stream(device=dev)
    sp = stream.cuda_stream

    def parallel():
        lp.lp_layer_parallel_step(h, s["images"], s["x"][1:], s["labels"], s["kappa"], rho, s["loss"], s["dx"], lr,
                                  0.0, 0.0, rho, sp)

    def parallel_distill():
        parallel()
        if K > 1:
            lp.lp_auxnet_distill(h, s["images"], s["x"][1:], s["dx"], lr, lr, None, s["dloss"], sp)

    def serial():
        lp.lp_serial_fwd_bwd(h, s["images"], s["labels"], s["loss"][K - 1], sp)
        lp.lp_step(h, lr, 0.0, 0.0, 0.0, None, sp)

    def one_after_another():
        lp.lp_auxnet_forward(h, s["images"], s["x"][1:], sp)
        for k in range(K):
            last = k == K - 1
            lp.lp_module_fwd_bwd(h, k, s["x"][k], s["labels"] if last else s["x"][k + 1],
                                 None if (last or s["kappa"] is None) else s["kappa"][k], rho, s["loss"][k],
                                 s["dx"][k], sp)
        lp.lp_step(h, lr, 0.0, 0.0, rho, s["kappa"], sp)
        if K > 1:
            lp.lp_auxnet_distill(h, s["images"], s["x"][1:], s["dx"], lr, lr, None, s["dloss"], sp)

    with torch.cuda.stream(stream):
        t_par = _time_graph(lp, torch, s, parallel, stream, reps)
        t_par_d = _time_graph(lp, torch, s, parallel_distill, stream, reps) if K > 1 else t_par
        t_ser = _time_graph(lp, torch, s, serial, stream, reps)
        for _ in range(2):
            one_after_another()
        torch.cuda.synchronize()
        lp.lp_timeline(h, True, read=False)
        one_after_another()
        recs = lp.lp_timeline(h, False)
    lp.lp_destroy(h)

    def total(pred):
        return sum(r["end_ms"] - r["start_ms"] for r in recs if pred(r))
    T_f = total(lambda r: r["phase"] == "forward" and r["op"] != "out_loss")
    T_b = total(lambda r: r["phase"] in ("backward", "update"))
    t_psi = total(lambda r: r["op"] == "out_loss")
    t_fl = total(lambda r: r["phase"] == "aux_forward")
    t_bl = total(lambda r: r["phase"] == "distill")
    overhead = t_psi + t_fl + t_bl
    N = cfg["N"]
    return {"workload": workload, "K": K, "batch": N, "module_block_end": cfg["module_block_end"],
            "phases_ms": {"T_f": T_f, "T_b": T_b, "t_psi": t_psi, "t_f_lambda": t_fl, "t_b_lambda": t_bl},
            "step_ms": {"layer_serial": t_ser, "layer_parallel": t_par, "layer_parallel_with_distillation": t_par_d},
            "images_per_s": {"layer_serial": N / t_ser * 1e3, "layer_parallel": N / t_par * 1e3,
                             "layer_parallel_with_distillation": N / t_par_d * 1e3},
            "rho_model_K_devices": 1.0 / (1.0 / K + overhead / (T_f + T_b)),
            "rho_model_upper_bound": (T_f + T_b) / overhead if overhead > 0 else None,
            "rho_measured_one_gpu": t_ser / t_par, "rho_measured_one_gpu_with_distillation": t_ser / t_par_d}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="wrn28_10")
    ap.add_argument("--K", type=int, nargs="+", default=[1, 2, 3, 4, 6])
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--reps", type=int, default=30)
    a = ap.parse_args()
    for K in a.K:
        print(json.dumps(measure(a.workload, K, a.batch, a.reps)), flush=True)


if __name__ == "__main__":
    main()
