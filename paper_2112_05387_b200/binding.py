"""ctypes binding with the same names as the C ABI in include/lp.h (argument marshalling only)."""
import ctypes
import os

import numpy as np

__all__ = [
    "LP_OK", "LP_F32", "LP_BF16", "LP_AUX", "LP_REAUX", "LP_CONV_IMPL_AUTO", "LP_CONV_IMPL_SIMT", "LP_CONV_IMPL_TENSOR", "LP_CONV_LOSS_IN_EPILOGUE", "LP_CONV_DIRECT_EPILOGUE", "LP_CONV_STAGED_EPILOGUE", "LP_CONV_TWO_CTA", "LP_CONV_BN_REDUCE_IN_EPILOGUE", "LP_CONV_WGRAD_IN_CHAIN",
    "LP_CONV_FWD", "LP_CONV_DGRAD", "LP_CONV_WGRAD", "LpError", "lp_net_desc", "lp_param_entry", "library",
    "library_path", "desc_from_config", "lp_status_string", "lp_validate_desc", "lp_workspace_bytes",
    "lp_param_layout", "lp_boundary_shape_desc", "lp_create", "lp_destroy", "lp_param_count", "lp_set_params",
    "lp_get_params", "lp_get_grads", "lp_boundary_shape", "lp_auxnet_forward", "lp_module_fwd_bwd",
    "lp_modules_fwd_bwd_all", "lp_step", "lp_forward_serial", "lp_serial_fwd_bwd", "lp_get_residual",
    "lp_last_device_status", "lp_launch_count", "lp_conv_profile", "lp_conv2d", "lp_conv2d_scratch_bytes", "lp_graph_begin", "lp_graph_end",
    "lp_graph_launch", "lp_conv2d_fwd_noalloc", "LP_NOALLOC_SCRATCH_BYTES", "lp_layer_parallel_step", "lp_auxnet_distill", "lp_aux_correct", "lp_timeline", "lp_timeline_record",
    "LP_PHASE_NAMES", "LP_OP_NAMES", "EXPORTED_SYMBOLS", "lp_selftest_bounded_wait",
]

LP_OK = 0
LP_F32, LP_BF16 = 0, 1
LP_CONV_IMPL_AUTO, LP_CONV_IMPL_SIMT, LP_CONV_IMPL_TENSOR = 0, 1, 2
LP_CONV_LOSS_IN_EPILOGUE = 128
LP_CONV_DIRECT_EPILOGUE, LP_CONV_STAGED_EPILOGUE = 256, 512
LP_CONV_TWO_CTA = 1024
LP_CONV_BN_REDUCE_IN_EPILOGUE = 2048
LP_CONV_WGRAD_IN_CHAIN = 4096
LP_CONV_FWD, LP_CONV_DGRAD, LP_CONV_WGRAD = 0, 1, 2
LP_MAX_STAGES, LP_MAX_MODULES = 8, 16
LP_NOALLOC_SCRATCH_BYTES = 8 << 20
_KINDS = ["conv_w", "bn_gamma", "bn_beta", "fc_w", "fc_b"]
LP_PHASE_NAMES = ["aux_forward", "forward", "backward", "update", "distill"]
LP_OP_NAMES = ["conv_fwd", "conv_dgrad", "conv_wgrad", "bn_stats", "bn_apply", "out_loss", "bn_bwd", "maxpool_fwd",
               "maxpool_bwd", "head_fwd", "head_bwd", "copy", "update"]

EXPORTED_SYMBOLS = [
    "lp_status_string", "lp_workspace_bytes", "lp_validate_desc", "lp_param_layout", "lp_boundary_shape_desc",
    "lp_create", "lp_destroy", "lp_param_count", "lp_set_params", "lp_get_params", "lp_get_grads",
    "lp_boundary_shape", "lp_auxnet_forward", "lp_module_fwd_bwd", "lp_modules_fwd_bwd_all", "lp_step",
    "lp_forward_serial", "lp_serial_fwd_bwd", "lp_get_residual", "lp_last_device_status", "lp_launch_count",
    "lp_conv_profile", "lp_conv2d_scratch_bytes", "lp_conv2d", "lp_graph_begin", "lp_graph_end", "lp_graph_launch",
    "lp_conv2d_fwd_noalloc", "lp_layer_parallel_step", "lp_auxnet_distill", "lp_timeline", "lp_aux_correct",
    "lp_selftest_bounded_wait",
]


def LP_AUX(k):
    return 256 + k


def LP_REAUX(k, j):
    """Unit j (0 <= j < k) of the recursive stack that generates x_k (descriptor aux_recursive = 1)."""
    return LP_AUX(k * (k - 1) // 2 + j)


class LpError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, lp_status_string(status), status))


class lp_net_desc(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("dtype", ctypes.c_int32),
        ("N", ctypes.c_int32), ("H", ctypes.c_int32), ("W", ctypes.c_int32), ("C_in", ctypes.c_int32),
        ("num_classes", ctypes.c_int32), ("stem_kind", ctypes.c_int32), ("stem_channels", ctypes.c_int32),
        ("block_kind", ctypes.c_int32), ("post_add_relu", ctypes.c_int32), ("num_stages", ctypes.c_int32),
        ("stage_channels", ctypes.c_int32 * LP_MAX_STAGES), ("stage_blocks", ctypes.c_int32 * LP_MAX_STAGES),
        ("stage_stride", ctypes.c_int32 * LP_MAX_STAGES), ("K", ctypes.c_int32),
        ("module_block_end", ctypes.c_int32 * LP_MAX_MODULES), ("aux_convs_per_boundary", ctypes.c_int32),
        ("aux_width_div", ctypes.c_int32), ("bn_eps", ctypes.c_float), ("conv_impl", ctypes.c_int32), ("aux_recursive", ctypes.c_int32),
    ]


class lp_param_entry(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 48), ("kind", ctypes.c_int32), ("shape", ctypes.c_int32 * 4),
                ("offset", ctypes.c_uint64)]


class lp_timeline_record(ctypes.Structure):
    _fields_ = [("plan", ctypes.c_int32), ("op", ctypes.c_int32), ("phase", ctypes.c_int32),
                ("start_ms", ctypes.c_float), ("end_ms", ctypes.c_float), ("bytes", ctypes.c_double)]


_LIB = None


def library_path():
    """In-tree liblp.so, or the library named by LP_LIBRARY_PATH (for trying out a different build)."""
    return os.environ.get("LP_LIBRARY_PATH") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblp.so")


def library():
    """Load liblp.so (built in-tree by __graft_entry__.build()); there is no fallback path."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError("liblp.so is not built: run `python -c 'import __graft_entry__ as g; g.build()'`")
    lib = ctypes.CDLL(path)
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    dp = ctypes.POINTER(lp_net_desc)
    lib.lp_status_string.restype = ctypes.c_char_p
    lib.lp_status_string.argtypes = [i32]
    lib.lp_workspace_bytes.restype = sz
    lib.lp_workspace_bytes.argtypes = [dp]
    lib.lp_validate_desc.argtypes = [dp]
    lib.lp_param_layout.argtypes = [dp, i32, ctypes.POINTER(lp_param_entry), i32, ctypes.POINTER(i32)]
    lib.lp_boundary_shape_desc.argtypes = [dp, i32, ctypes.POINTER(i32 * 4)]
    lib.lp_create.argtypes = [dp, vp, sz, ctypes.POINTER(vp)]
    lib.lp_destroy.argtypes = [vp]
    lib.lp_param_count.argtypes = [vp, i32, ctypes.POINTER(sz)]
    lib.lp_set_params.argtypes = [vp, i32, vp, sz]
    lib.lp_get_params.argtypes = [vp, i32, vp, sz]
    lib.lp_get_grads.argtypes = [vp, i32, vp, sz]
    lib.lp_boundary_shape.argtypes = [vp, i32, ctypes.POINTER(i32 * 4)]
    lib.lp_auxnet_forward.argtypes = [vp, vp, ctypes.POINTER(vp), vp]
    lib.lp_module_fwd_bwd.argtypes = [vp, i32, vp, vp, vp, f32, vp, vp, vp]
    lib.lp_modules_fwd_bwd_all.argtypes = [vp, ctypes.POINTER(vp), vp, ctypes.POINTER(vp), f32, vp,
                                           ctypes.POINTER(vp), vp]
    lib.lp_step.argtypes = [vp, f32, f32, f32, f32, ctypes.POINTER(vp), vp]
    lib.lp_layer_parallel_step.argtypes = [vp, vp, ctypes.POINTER(vp), vp, ctypes.POINTER(vp), f32, vp,
                                           ctypes.POINTER(vp), f32, f32, f32, f32, vp]
    lib.lp_auxnet_distill.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), f32, f32, ctypes.POINTER(vp), vp, vp]
    lib.lp_aux_correct.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), f32, vp, vp]
    lib.lp_aux_correct.restype = i32
    lib.lp_forward_serial.argtypes = [vp, vp, vp, vp]
    lib.lp_serial_fwd_bwd.argtypes = [vp, vp, vp, vp, vp]
    lib.lp_get_residual.argtypes = [vp, i32, vp, vp, vp]
    lib.lp_last_device_status.argtypes = [vp, vp]
    lib.lp_selftest_bounded_wait.argtypes = [vp, ctypes.c_double, ctypes.POINTER(ctypes.c_double), vp]
    lib.lp_launch_count.restype = ctypes.c_int64
    lib.lp_launch_count.argtypes = [vp, i32]
    lib.lp_timeline.argtypes = [vp, i32, i32, ctypes.POINTER(lp_timeline_record), ctypes.POINTER(ctypes.c_int)]
    lib.lp_timeline.restype = i32
    lib.lp_conv_profile.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                    ctypes.POINTER(ctypes.c_int64)]
    lib.lp_graph_begin.argtypes = [vp, vp]
    lib.lp_graph_end.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.lp_graph_launch.argtypes = [vp, i32, vp]
    lib.lp_conv2d_fwd_noalloc.argtypes = [i32] * 8 + [vp, vp, vp, vp]
    lib.lp_conv2d_scratch_bytes.restype = sz
    lib.lp_conv2d_scratch_bytes.argtypes = [i32, i32, i32]
    lib.lp_conv2d.argtypes = [i32] * 11 + [vp, vp, vp, vp, vp, sz, ctypes.POINTER(f32), vp]
    _LIB = lib
    return lib


def _ptr(t):
    """Raw address of a torch tensor / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _check(status, where):
    if status != LP_OK:
        raise LpError(status, where)


def desc_from_config(cfg, conv_impl=LP_CONV_IMPL_AUTO, aux_recursive=False):
    """Translate a workload dict (workloads/configs.py) into the C descriptor."""
    d = lp_net_desc()
    d.struct_size = ctypes.sizeof(lp_net_desc)
    d.dtype = LP_F32 if cfg["dtype"] == "f32" else LP_BF16
    d.N, d.H, d.W, d.C_in = cfg["N"], cfg["H"], cfg["W"], cfg["C_in"]
    d.num_classes = cfg["num_classes"]
    d.stem_kind = 0 if cfg["stem_kind"] == "conv3x3" else 1
    d.stem_channels = cfg["stem_channels"]
    d.block_kind = {"postbn": 0, "preact": 1, "bottleneck": 2}[cfg["block_kind"]]
    d.post_add_relu = 0
    d.num_stages = len(cfg["stage_channels"])
    for i, (c, b, s) in enumerate(zip(cfg["stage_channels"], cfg["stage_blocks"], cfg["stage_stride"])):
        d.stage_channels[i], d.stage_blocks[i], d.stage_stride[i] = c, b, s
    d.K = len(cfg["module_block_end"])
    for i, e in enumerate(cfg["module_block_end"]):
        d.module_block_end[i] = e
    d.aux_convs_per_boundary = cfg["aux_convs"]
    d.aux_width_div = cfg["aux_width_div"]
    d.bn_eps = cfg["bn_eps"]
    d.conv_impl = conv_impl
    d.aux_recursive = 1 if aux_recursive else 0
    return d


def lp_status_string(status):
    return library().lp_status_string(status).decode()


def lp_validate_desc(desc):
    return library().lp_validate_desc(ctypes.byref(desc))


def lp_workspace_bytes(desc):
    return library().lp_workspace_bytes(ctypes.byref(desc))


def lp_param_layout(desc, which):
    """List of (name, kind, shape) in blob order, the same form the oracle reports."""
    n = ctypes.c_int(0)
    _check(library().lp_param_layout(ctypes.byref(desc), which, None, 0, ctypes.byref(n)), "lp_param_layout")
    arr = (lp_param_entry * n.value)()
    _check(library().lp_param_layout(ctypes.byref(desc), which, arr, n.value, ctypes.byref(n)), "lp_param_layout")
    return [(e.name.decode(), _KINDS[e.kind], tuple(int(s) for s in e.shape if s > 0)) for e in arr]


def lp_boundary_shape_desc(desc, k):
    s = (ctypes.c_int * 4)()
    _check(library().lp_boundary_shape_desc(ctypes.byref(desc), k, ctypes.byref(s)), "lp_boundary_shape_desc")
    return tuple(s)


class Handle:
    """An lp_handle* together with the torch tensor that backs its workspace."""

    def __init__(self, ptr, workspace, desc):
        self.ptr, self.workspace, self.desc = ptr, workspace, desc
        self.K = desc.K

    def __del__(self):
        try:
            if self.ptr:
                library().lp_destroy(self.ptr)
                self.ptr = None
        except Exception:
            pass


def lp_create(desc, device="cuda:0"):
    """Allocate the workspace with torch (device memory only) and create the handle."""
    import torch
    need = lp_workspace_bytes(desc)
    if need == 0:
        raise LpError(lp_validate_desc(desc) or -2, "lp_workspace_bytes")
    ws = torch.empty(need + 256, dtype=torch.uint8, device=device)
    base = (ws.data_ptr() + 255) // 256 * 256
    out = ctypes.c_void_p()
    _check(library().lp_create(ctypes.byref(desc), base, need, ctypes.byref(out)), "lp_create")
    return Handle(out.value, ws, desc)


def lp_destroy(h):
    if h.ptr:
        _check(library().lp_destroy(h.ptr), "lp_destroy")
        h.ptr = None


def lp_param_count(h, which):
    n = ctypes.c_size_t(0)
    _check(library().lp_param_count(h.ptr, which, ctypes.byref(n)), "lp_param_count")
    return n.value


def lp_set_params(h, which, host_array):
    a = np.ascontiguousarray(host_array, dtype=np.float32)
    _check(library().lp_set_params(h.ptr, which, a.ctypes.data, a.size), "lp_set_params")


def lp_get_params(h, which):
    a = np.empty(lp_param_count(h, which), dtype=np.float32)
    _check(library().lp_get_params(h.ptr, which, a.ctypes.data, a.size), "lp_get_params")
    return a


def lp_get_grads(h, which):
    a = np.empty(lp_param_count(h, which), dtype=np.float32)
    _check(library().lp_get_grads(h.ptr, which, a.ctypes.data, a.size), "lp_get_grads")
    return a


def lp_boundary_shape(h, k):
    s = (ctypes.c_int * 4)()
    _check(library().lp_boundary_shape(h.ptr, k, ctypes.byref(s)), "lp_boundary_shape")
    return tuple(s)


def _ptr_array(items, n):
    arr = (ctypes.c_void_p * max(n, 1))()
    for i in range(n):
        arr[i] = _ptr(items[i]) if items is not None and i < len(items) else None
    return arr


def lp_auxnet_forward(h, images, x_out, stream=None):
    arr = _ptr_array(x_out, h.K - 1)
    _check(library().lp_auxnet_forward(h.ptr, _ptr(images), arr, _ptr(stream)), "lp_auxnet_forward")


def lp_module_fwd_bwd(h, k, x_k, x_next_or_labels, lambda_k, rho, loss_out, dx_k, stream=None):
    _check(library().lp_module_fwd_bwd(h.ptr, k, _ptr(x_k), _ptr(x_next_or_labels), _ptr(lambda_k), rho,
                                       _ptr(loss_out), _ptr(dx_k), _ptr(stream)), "lp_module_fwd_bwd")


def lp_modules_fwd_bwd_all(h, x, labels, lambdas, rho, loss_out, dx, stream=None):
    xa = _ptr_array(x, h.K)
    la = _ptr_array(lambdas, h.K) if lambdas is not None else None
    da = _ptr_array(dx, h.K) if dx is not None else None
    _check(library().lp_modules_fwd_bwd_all(h.ptr, xa, _ptr(labels), la, rho, _ptr(loss_out), da, _ptr(stream)),
           "lp_modules_fwd_bwd_all")


def lp_step(h, lr, momentum=0.0, weight_decay=0.0, kappa_step=0.0, lambdas_inout=None, stream=None):
    la = _ptr_array(lambdas_inout, h.K) if lambdas_inout is not None else None
    _check(library().lp_step(h.ptr, lr, momentum, weight_decay, kappa_step, la, _ptr(stream)), "lp_step")


def lp_layer_parallel_step(h, images, x_out, labels, lambdas_inout, rho, loss_out, dx, lr, momentum=0.0,
                           weight_decay=0.0, kappa_step=0.0, stream=None):
    xa = _ptr_array(x_out, h.K - 1)
    la = _ptr_array(lambdas_inout, h.K) if lambdas_inout is not None else None
    da = _ptr_array(dx, h.K) if dx is not None else None
    _check(library().lp_layer_parallel_step(h.ptr, _ptr(images), xa, _ptr(labels), la, rho, _ptr(loss_out), da, lr,
                                            momentum, weight_decay, kappa_step, _ptr(stream)),
           "lp_layer_parallel_step")


def lp_auxnet_distill(h, images, x, dx, lr_lambda, lr_aux, x_new, loss_out, stream=None):
    xa = _ptr_array(x, h.K - 1)
    da = _ptr_array(dx, h.K)
    na = _ptr_array(x_new, h.K - 1) if x_new is not None else None
    _check(library().lp_auxnet_distill(h.ptr, _ptr(images), xa, da, lr_lambda, lr_aux, na, _ptr(loss_out), _ptr(stream)),
           "lp_auxnet_distill")


def lp_aux_correct(h, x_inout, dx, lr_lambda, norm_out=None, stream=None):
    xa = _ptr_array(x_inout, h.K - 1)
    da = _ptr_array(dx, h.K)
    _check(library().lp_aux_correct(h.ptr, xa, da, lr_lambda, _ptr(norm_out), _ptr(stream)), "lp_aux_correct")


def lp_forward_serial(h, images, logits, stream=None):
    _check(library().lp_forward_serial(h.ptr, _ptr(images), _ptr(logits), _ptr(stream)), "lp_forward_serial")


def lp_serial_fwd_bwd(h, images, labels, loss_out, stream=None):
    _check(library().lp_serial_fwd_bwd(h.ptr, _ptr(images), _ptr(labels), _ptr(loss_out), _ptr(stream)),
           "lp_serial_fwd_bwd")


def lp_get_residual(h, k, r_dst, seed_dst, stream=None):
    _check(library().lp_get_residual(h.ptr, k, _ptr(r_dst), _ptr(seed_dst), _ptr(stream)), "lp_get_residual")


def lp_last_device_status(h, stream=None):
    return library().lp_last_device_status(h.ptr, _ptr(stream))


def lp_selftest_bounded_wait(h, limit_ms, stream=None):
    """Launch the bounded-wait self-test; returns the milliseconds the device thread waited before giving up."""
    w = ctypes.c_double(0.0)
    _check(library().lp_selftest_bounded_wait(h.ptr, float(limit_ms), ctypes.byref(w), _ptr(stream)),
           "lp_selftest_bounded_wait")
    return w.value


def lp_launch_count(h, reset=False):
    return int(library().lp_launch_count(h.ptr, 1 if reset else 0))


def lp_conv_profile(h, enable, read=True):
    ms, fl, n = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_int64(0)
    if read:
        _check(library().lp_conv_profile(h.ptr, 1 if enable else 0, ctypes.byref(ms), ctypes.byref(fl),
                                         ctypes.byref(n)), "lp_conv_profile")
    else:
        _check(library().lp_conv_profile(h.ptr, 1 if enable else 0, None, None, None), "lp_conv_profile")
    return ms.value, fl.value, n.value


def lp_timeline(h, enable, read=True, max_records=4096):
    """Enable/disable the per-operation time line; with ``read`` returns the records collected so far
    as a list of dicts (plan, op, phase, start_ms, end_ms)."""
    if not read:
        _check(library().lp_timeline(h.ptr, 1 if enable else 0, 0, None, None), "lp_timeline")
        return []
    recs = (lp_timeline_record * max_records)()
    n = ctypes.c_int(0)
    _check(library().lp_timeline(h.ptr, 1 if enable else 0, max_records, recs, ctypes.byref(n)), "lp_timeline")
    return [dict(plan=r.plan, op=LP_OP_NAMES[r.op], phase=LP_PHASE_NAMES[r.phase], start_ms=r.start_ms, end_ms=r.end_ms,
                 bytes=r.bytes)
            for r in recs[:min(n.value, max_records)]]


def lp_graph_begin(h, stream):
    _check(library().lp_graph_begin(h.ptr, _ptr(stream)), "lp_graph_begin")


def lp_graph_end(h, stream):
    gid = ctypes.c_int(-1)
    _check(library().lp_graph_end(h.ptr, _ptr(stream), ctypes.byref(gid)), "lp_graph_end")
    return gid.value


def lp_graph_launch(h, graph_id, stream=None):
    _check(library().lp_graph_launch(h.ptr, graph_id, _ptr(stream)), "lp_graph_launch")


def lp_conv2d_scratch_bytes(cin, cout, r):
    return library().lp_conv2d_scratch_bytes(cin, cout, r)


def lp_conv2d(op, dtype, impl, N, H, W, Cin, Cout, R, stride, pad, a, b, out, stats, scratch, scratch_bytes,
              timed=False, stream=None):
    """Returns (status, elapsed_ms or None)."""
    ms = ctypes.c_float(0.0)
    st = library().lp_conv2d(op, dtype, impl, N, H, W, Cin, Cout, R, stride, pad, _ptr(a), _ptr(b), _ptr(out),
                             _ptr(stats), _ptr(scratch), scratch_bytes, ctypes.byref(ms) if timed else None,
                             _ptr(stream))
    return st, (ms.value if timed else None)


def lp_conv2d_fwd_noalloc(N, H, W, Cin, Cout, R, stride, pad, x, w, y, stream=None):
    """Forward convolution whose scratch is a fixed array inside the library: for callers that may
    not allocate device memory.  Returns the status (0 = ok); see include/lp.h for the limits."""
    return library().lp_conv2d_fwd_noalloc(N, H, W, Cin, Cout, R, stride, pad, _ptr(x), _ptr(w), _ptr(y), _ptr(stream))
