"""ctypes binding of include/asteroid.h: same names, argument marshalling only."""
import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libasteroid.so")

AST_F32, AST_BF16 = 0, 1
AST_OK, AST_ERR_ARG, AST_ERR_UNSUPPORTED, AST_ERR_ORDER, AST_ERR_ALLOC, AST_ERR_CUDA, AST_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
OP_CODES = {"conv": 0, "dwconv": 1, "bn": 2, "relu6": 3, "relu": 4, "add": 5, "gap": 6, "linear": 7, "silu": 8, "se": 9}

EXPORTS = ["asteroid_stage_create", "asteroid_stage_destroy", "asteroid_stage_param_count",
           "asteroid_stage_output_elems", "asteroid_stage_import_state", "asteroid_stage_export_state",
           "asteroid_stage_export_bn_running", "asteroid_stage_forward", "asteroid_stage_backward",
           "asteroid_stage_accumulate", "asteroid_stage_step", "asteroid_stage_grad_buffer", "asteroid_stage_profile",
           "asteroid_loss_mse", "asteroid_loss_mse_noalloc", "asteroid_loss_softmax_xent", "asteroid_trace_start", "asteroid_trace_stop",
           "asteroid_selftest_bounded_wait", "asteroid_plan", "asteroid_launch_count", "asteroid_last_error"]


class ast_layer(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("op", "c_in", "c_out", "k", "stride", "pad", "src", "add_from")]


class ast_opts(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("slots", C.c_int32), ("need_input_grad", C.c_int32),
                ("bn_eps", C.c_float), ("bn_momentum", C.c_float)]


class ast_layer_profile(C.Structure):
    _fields_ = [("t_f_ms", C.c_double), ("t_b_ms", C.c_double)] + \
               [(n, C.c_uint64) for n in ("a_l_bytes", "w_l_bytes", "flops", "alg_bytes_f", "alg_bytes_b",
                                          "mem_mod", "mem_opt", "mem_act", "mem_work")] + \
               [("fused_into", C.c_int32), ("reserved", C.c_int32)]


class ast_kernel_stat(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_uint64), ("total_ms", C.c_double),
                ("alg_bytes", C.c_double), ("flops", C.c_double)]


PLAN_MAX_DEVICES = 64


class ast_plan_problem(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "n_types", "n_bs", "N", "B", "M", "block")] + \
               [("bs", C.POINTER(C.c_int32)), ("t_f", C.POINTER(C.c_double)), ("t_b", C.POINTER(C.c_double)),
                ("a", C.POINTER(C.c_double)), ("w", C.POINTER(C.c_double)), ("act", C.POINTER(C.c_double)),
                ("mod_factor", C.c_double), ("opt_factor", C.c_double), ("dev_type", C.POINTER(C.c_int32)),
                ("dev_mem", C.POINTER(C.c_double)), ("bw", C.POINTER(C.c_double))]


class ast_plan_result(C.Structure):
    _fields_ = [("latency_ms", C.c_double), ("n_stages", C.c_int32), ("n_steps", C.c_int32), ("dominant_step", C.c_int32), ("reserved", C.c_int32),
                ("first_layer", C.c_int32 * PLAN_MAX_DEVICES), ("last_layer", C.c_int32 * PLAN_MAX_DEVICES), ("dev_begin", C.c_int32 * (PLAN_MAX_DEVICES + 1)),
                ("devices", C.c_int32 * PLAN_MAX_DEVICES), ("samples", C.c_int32 * PLAN_MAX_DEVICES),
                ("e_f_ms", C.c_double * PLAN_MAX_DEVICES), ("e_b_ms", C.c_double * PLAN_MAX_DEVICES), ("t_a_ms", C.c_double * PLAN_MAX_DEVICES)]


class AsteroidError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("asteroid error %d: %s" % (code, msg))
        self.code = code


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("%s is missing: run `python -m paper_2408_08015_b200.build` (needs nvcc)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
        fp = C.POINTER(C.c_float)
        L.asteroid_stage_create.argtypes = [C.POINTER(ast_layer), i, i, i, i, i, i, i, C.POINTER(ast_opts), C.POINTER(vp)]
        L.asteroid_stage_destroy.argtypes = [vp]
        L.asteroid_stage_destroy.restype = None
        L.asteroid_stage_param_count.argtypes = [vp]
        L.asteroid_stage_param_count.restype = sz
        L.asteroid_stage_output_elems.argtypes = [vp, C.POINTER(i), C.POINTER(i), C.POINTER(i)]
        L.asteroid_stage_output_elems.restype = sz
        L.asteroid_stage_import_state.argtypes = [vp, fp, fp, sz]
        L.asteroid_stage_export_state.argtypes = [vp, fp, fp, fp, fp, sz]
        L.asteroid_stage_export_bn_running.argtypes = [vp, fp, fp, sz]
        L.asteroid_stage_forward.argtypes = [vp, i, vp, vp, vp]
        L.asteroid_stage_backward.argtypes = [vp, i, vp, vp, vp]
        L.asteroid_stage_accumulate.argtypes = [vp, i, vp]
        L.asteroid_stage_step.argtypes = [vp, f, f, vp]
        L.asteroid_stage_grad_buffer.argtypes = [vp, C.POINTER(vp), C.POINTER(sz)]
        L.asteroid_stage_profile.argtypes = [vp, i, i, C.POINTER(ast_layer_profile)]
        L.asteroid_loss_mse.argtypes = [vp, vp, sz, i, vp, vp, vp]
        L.asteroid_loss_mse_noalloc.argtypes = [vp, vp, sz, i, vp, vp, vp]
        L.asteroid_loss_softmax_xent.argtypes = [vp, vp, i, i, i, vp, vp, vp]
        L.asteroid_trace_start.argtypes = []
        L.asteroid_trace_stop.argtypes = [C.POINTER(ast_kernel_stat), i, C.POINTER(i)]
        L.asteroid_selftest_bounded_wait.argtypes = []
        L.asteroid_plan.argtypes = [C.POINTER(ast_plan_problem), C.POINTER(ast_plan_result)]
        L.asteroid_launch_count.argtypes = []
        L.asteroid_launch_count.restype = C.c_uint64
        L.asteroid_last_error.argtypes = []
        L.asteroid_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(rc):
    if rc != 0:
        raise AsteroidError(rc, lib().asteroid_last_error().decode())


def _fptr(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_float))


def pack_layers(net):
    """`net`: sequence of records with fields op (name or code), c_in, c_out, k, stride, pad, src, add_from."""
    arr = (ast_layer * len(net))()
    for j, l in enumerate(net):
        op = OP_CODES[l.op] if isinstance(l.op, str) else int(l.op)
        arr[j] = ast_layer(op, l.c_in, l.c_out, l.k, l.stride, l.pad, l.src, l.add_from)
    return arr


def asteroid_stage_create(net, first, last, in_h, in_w, micro_batch, M, dtype=AST_F32, slots=0,
                          need_input_grad=1, bn_eps=0.0, bn_momentum=0.0):
    arr = pack_layers(net)
    opts = ast_opts(dtype, slots, need_input_grad, bn_eps, bn_momentum)
    h = C.c_void_p()
    _check(lib().asteroid_stage_create(arr, len(net), first, last, in_h, in_w, micro_batch, M, C.byref(opts), C.byref(h)))
    return h


def asteroid_stage_destroy(h):
    lib().asteroid_stage_destroy(h)


def asteroid_stage_param_count(h):
    return lib().asteroid_stage_param_count(h)


def asteroid_stage_output_elems(h):
    a, b, c = C.c_int(), C.c_int(), C.c_int()
    n = lib().asteroid_stage_output_elems(h, C.byref(a), C.byref(b), C.byref(c))
    return n, (a.value, b.value, c.value)


def asteroid_stage_grad_buffer(h):
    """(device address, length in floats) of the stage's accumulated-gradient arena."""
    g, n = C.c_void_p(), C.c_size_t()
    _check(lib().asteroid_stage_grad_buffer(h, C.byref(g), C.byref(n)))
    return g.value, n.value


def asteroid_stage_import_state(h, params, momentum=None):
    """params / momentum: contiguous float32 numpy arrays (host)."""
    _check(lib().asteroid_stage_import_state(h, _fptr(params), _fptr(momentum), params.size))


def asteroid_stage_export_state(h, params=None, momentum=None, grad_accum=None, micro_grad=None):
    n = asteroid_stage_param_count(h)
    _check(lib().asteroid_stage_export_state(h, _fptr(params), _fptr(momentum), _fptr(grad_accum), _fptr(micro_grad), n))


def asteroid_stage_export_bn_running(h, mean, var):
    _check(lib().asteroid_stage_export_bn_running(h, _fptr(mean), _fptr(var), mean.size))


def asteroid_stage_forward(h, mb, x_ptr, y_ptr, stream=0):
    _check(lib().asteroid_stage_forward(h, mb, x_ptr, y_ptr, stream))


def asteroid_stage_backward(h, mb, dy_ptr, dx_ptr, stream=0):
    _check(lib().asteroid_stage_backward(h, mb, dy_ptr, dx_ptr, stream))


def asteroid_stage_accumulate(h, mb, stream=0):
    _check(lib().asteroid_stage_accumulate(h, mb, stream))


def asteroid_stage_step(h, lr, momentum, stream=0):
    _check(lib().asteroid_stage_step(h, lr, momentum, stream))


def asteroid_stage_profile(h, layer, batch):
    rec = ast_layer_profile()
    _check(lib().asteroid_stage_profile(h, layer, batch, C.byref(rec)))
    return {n: getattr(rec, n) for n, _ in ast_layer_profile._fields_ if n != "reserved"}


def asteroid_loss_mse(y_ptr, t_ptr, n, dtype, dy_ptr, loss_ptr, stream=0):
    _check(lib().asteroid_loss_mse(y_ptr, t_ptr, n, dtype, dy_ptr, loss_ptr, stream))


def asteroid_loss_mse_noalloc(y_ptr, t_ptr, n, dtype, dy_ptr, loss_ptr, stream=0):
    """MSE head that performs no device allocation (static scratch inside the library; n <= 2**26)."""
    _check(lib().asteroid_loss_mse_noalloc(y_ptr, t_ptr, n, dtype, dy_ptr, loss_ptr, stream))


def asteroid_loss_softmax_xent(logits_ptr, labels_ptr, rows, classes, dtype, dlogits_ptr, loss_ptr, stream=0):
    _check(lib().asteroid_loss_softmax_xent(logits_ptr, labels_ptr, rows, classes, dtype, dlogits_ptr, loss_ptr, stream))


def asteroid_trace_start():
    _check(lib().asteroid_trace_start())


def asteroid_trace_stop():
    """[{name, launches, total_ms, alg_bytes, flops}] per kernel kind that ran since trace_start."""
    buf = (ast_kernel_stat * 64)()
    n = C.c_int()
    _check(lib().asteroid_trace_stop(buf, 64, C.byref(n)))
    return [{"name": buf[j].name.decode(), "launches": buf[j].launches, "total_ms": buf[j].total_ms,
             "alg_bytes": buf[j].alg_bytes, "flops": buf[j].flops} for j in range(n.value)]


def asteroid_selftest_bounded_wait():
    """Return code of the bounded-wait self-test (AST_ERR_TIMEOUT is the expected outcome); does not raise."""
    return lib().asteroid_selftest_bounded_wait()


def asteroid_plan(prob):
    """`prob`: the dict form of a planning problem (keys L, B, M, block, bs, t_f[type][l][k], t_b, a, w, act, mod_factor, opt_factor,
    devices [{type, mem}], bw[d][d']).  Returns {"latency", "dm", "stages": [{"layers": (i, j), "devices": [...], "y": [...],
    "ef", "eb", "ta"}]} or None when nothing fits.  Marshalling only: the planning runs in the library."""
    import numpy as np
    L, N = int(prob["L"]), len(prob["devices"])
    bs = np.ascontiguousarray(prob["bs"], np.int32)
    tf = np.ascontiguousarray(prob["t_f"], np.float64)
    tb = np.ascontiguousarray(prob["t_b"], np.float64)
    a, w, act = (np.ascontiguousarray(prob[k], np.float64) for k in ("a", "w", "act"))
    dt = np.ascontiguousarray([d["type"] for d in prob["devices"]], np.int32)
    dm = np.ascontiguousarray([d["mem"] for d in prob["devices"]], np.float64)
    bw = np.ascontiguousarray(prob["bw"], np.float64)
    dp, ip = (lambda x: x.ctypes.data_as(C.POINTER(C.c_double))), (lambda x: x.ctypes.data_as(C.POINTER(C.c_int32)))
    p = ast_plan_problem(L, tf.shape[0], bs.size, N, int(prob["B"]), int(prob["M"]), int(prob["block"]), ip(bs), dp(tf), dp(tb), dp(a), dp(w), dp(act),
                         float(prob["mod_factor"]), float(prob["opt_factor"]), ip(dt), dp(dm), dp(bw))
    r = ast_plan_result()
    _check(lib().asteroid_plan(C.byref(p), C.byref(r)))
    if r.n_stages == 0:
        return None
    stages = []
    for s in range(r.n_stages):
        q0, q1 = r.dev_begin[s], r.dev_begin[s + 1]
        stages.append({"layers": (r.first_layer[s], r.last_layer[s]), "devices": list(r.devices[q0:q1]), "y": list(r.samples[q0:q1]),
                       "ef": r.e_f_ms[s], "eb": r.e_b_ms[s], "ta": r.t_a_ms[s]})
    return {"latency": r.latency_ms, "dm": r.dominant_step, "n_steps": r.n_steps, "stages": stages}


def asteroid_launch_count():
    return lib().asteroid_launch_count()


def asteroid_last_error():
    return lib().asteroid_last_error().decode()
