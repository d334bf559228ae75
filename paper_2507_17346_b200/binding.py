"""ctypes binding of libdeco: one Python function per C entry point, same names.

Argument marshalling only — every step of the path runs in the library's CUDA kernels.
Tensors are passed as raw device pointers (``tensor.data_ptr()``) and the current PyTorch
stream's handle; PyTorch is used for device memory and streams, nothing else.  There is no
fallback: if ``libdeco.so`` is missing or no CUDA device is present the calls raise.
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# DECO_LIB names another build of the library (for instance a debug build); default: in-tree.
LIB_PATH = os.environ.get("DECO_LIB") or os.path.join(_HERE, "libdeco.so")

DECO_OK = 0
DECO_ERR_INVALID_ARG = 1
DECO_ERR_OOM = 2
DECO_ERR_CUDA = 3
DECO_ERR_STATE = 4
DECO_ERR_CAPACITY = 5
DECO_ERR_TIMEOUT = 6
DECO_ERR_DEVICE_CHECK = 7

DECO_F32 = 0
DECO_BF16 = 1
DECO_NO_INDEX = 0xFFFFFFFF
DECO_SELECT_AUTO = 0
DECO_SELECT_EXACT_PASSES = 1
DECO_COMPRESSOR_TOPK = 0
DECO_COMPRESSOR_RANDK = 1


class deco_pair(ctypes.Structure):
    _fields_ = [("idx", ctypes.c_uint32), ("val", ctypes.c_float)]


class deco_options(ctypes.Structure):
    _fields_ = [("grad_dtype", ctypes.c_int32),
                ("tau_max", ctypes.c_uint32),
                ("delta_max", ctypes.c_double),
                ("lr_at_server", ctypes.c_int32),
                ("params", ctypes.c_void_p),
                ("device", ctypes.c_int32),
                ("select_mode", ctypes.c_int32),
                ("compressor", ctypes.c_int32),
                ("seed_lo", ctypes.c_uint32),
                ("seed_hi", ctypes.c_uint32),
                ("n_total", ctypes.c_uint32),
                ("worker_base", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32 * 3)]


class deco_lut_entry(ctypes.Structure):
    _fields_ = [("a_bps", ctypes.c_double), ("delta", ctypes.c_double),
                ("tau", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


class deco_stats(ctypes.Structure):
    _fields_ = [("step", ctypes.c_uint64),
                ("k", ctypes.c_uint64),
                ("delta", ctypes.c_double),
                ("tau", ctypes.c_uint32),
                ("device_status", ctypes.c_uint32),
                ("exact_pass_workers", ctypes.c_uint64),
                ("cached_aggregates", ctypes.c_uint64),
                ("device_bytes", ctypes.c_uint64)]


class DecoError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s: %s (%d)" % (where, status_string(status), status))


_lib = None

_vp, _u64, _u32, _i32, _f32, _f64 = (ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32,
                                     ctypes.c_int32, ctypes.c_float, ctypes.c_double)
_P = ctypes.POINTER

# name -> (restype, argtypes); the list mirrors include/deco.h
SIGNATURES = {
    "deco_init": (_i32, [_P(_vp), _u64, _u32, _f64, _u32, _f32, _P(deco_options)]),
    "deco_destroy": (None, [_vp]),
    "deco_reset": (_i32, [_vp, _vp]),
    "deco_ef_compress": (_i32, [_vp, _vp, _vp]),
    "deco_aggregate_stale": (_i32, [_vp, _vp]),
    "deco_apply_update": (_i32, [_vp, _vp]),
    "deco_step": (_i32, [_vp, _vp, _vp]),
    "deco_join": (_i32, [_vp, _vp]),
    "deco_step_host": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "deco_set_policy": (_i32, [_vp, _f64, _u32]),
    "deco_set_lr": (_i32, [_vp, _f32]),
    "deco_policy_select": (_i32, [_f64, _f64, _f64, _f64, _u32, _i32, _P(_u32), _P(_f64)]),
    "deco_lut_build": (_i32, [_f64, _f64, _f64, _f64, _f64, _u32, _u32, _i32,
                              _P(deco_lut_entry)]),
    "deco_lut_lookup": (_i32, [_P(deco_lut_entry), _u32, _f64, _f64, _f64, _f64, _u32, _i32,
                               _P(_u32), _P(_f64)]),
    "deco_t_avg": (_f64, [_f64, _u32, _f64, _f64, _f64, _f64]),
    "deco_k_from_delta": (_u64, [_f64, _u64]),
    "deco_get_k": (_i32, [_vp, _P(_u64)]),
    "deco_get_buffers": (_i32, [_vp, _P(_vp), _P(_u64), _P(_vp), _P(_u64), _P(_vp)]),
    "deco_get_aggregate": (_i32, [_vp, _u64, _P(_vp), _P(_u64)]),
    "deco_get_aggregate_vector": (_i32, [_vp, _u64, _P(_vp)]),
    "deco_get_select_info": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "deco_get_stats": (_i32, [_vp, _vp, _P(deco_stats)]),
    "deco_set_kernel_timing": (_i32, [_vp, _i32]),
    "deco_get_kernel_timing": (_i32, [_vp, _vp, _P(_f64), _P(_u64)]),
    "deco_state_bytes": (_i32, [_vp, _P(_u64)]),
    "deco_export_state": (_i32, [_vp, _vp, _u64, _vp]),
    "deco_import_state": (_i32, [_vp, _vp, _u64, _vp]),
    "deco_launch_count": (_u64, [_vp]),
    "deco_get_exchange": (_i32, [_vp, _P(_vp), _P(_u64), _P(_u32), _P(_u32), _P(_u32)]),
    "deco_topk_compress_static": (_i32, [_vp, _u64, _u64, _vp, _vp]),
    "deco_layered_init": (_i32, [_P(_vp), _u64, _u32, _P(_u64), _u32, _f64, _u32, _f32, _vp]),
    "deco_layered_destroy": (None, [_vp]),
    "deco_layered_step": (_i32, [_vp, _vp, _vp]),
    "deco_layered_join": (_i32, [_vp, _vp]),
    "deco_layered_set_policy": (_i32, [_vp, _f64, _u32]),
    "deco_layered_set_lr": (_i32, [_vp, _f32]),
    "deco_layered_layer": (_i32, [_vp, _u32, _P(_vp), _P(_u64), _P(_u64)]),
    "deco_layered_info": (_i32, [_vp, _P(_u32), _P(_u64), _P(_vp), _P(_u64)]),
    "deco_status_string": (ctypes.c_char_p, [_i32]),
}


def load():
    """Load libdeco.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError("libdeco.so not built: run `python -m paper_2507_17346_b200.build` "
                          "(expected at %s)" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def deco_status_string(status):
    return load().deco_status_string(int(status)).decode()


status_string = deco_status_string


def _check(status, where):
    if status != DECO_OK:
        raise DecoError(status, where)


def _ptr(x):
    """Raw address of a torch tensor / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ------------------------------------------------------------------ entry points

def _options(grad_dtype, tau_max, delta_max, lr_at_server, params, device, select_mode,
             compressor, seed, n_total=0, worker_base=0):
    opt = deco_options()
    opt.n_total = n_total
    opt.worker_base = worker_base
    opt.grad_dtype = grad_dtype
    opt.tau_max = tau_max
    opt.delta_max = delta_max
    opt.lr_at_server = int(bool(lr_at_server))
    opt.params = _ptr(params)
    opt.device = device
    opt.select_mode = select_mode
    opt.compressor = compressor
    opt.seed_lo = seed & 0xFFFFFFFF
    opt.seed_hi = (seed >> 32) & 0xFFFFFFFF
    return opt


def deco_init(d, n, delta, tau, lr, grad_dtype=DECO_F32, tau_max=0, delta_max=0.0,
              lr_at_server=False, params=None, device=0, select_mode=DECO_SELECT_AUTO,
              compressor=DECO_COMPRESSOR_TOPK, seed=0, n_total=0, worker_base=0):
    """-> opaque context handle (int).  `params`: optional fp32 CUDA tensor of length d.
    n_total / worker_base: this context holds n of the job's n_total workers (sharded job)."""
    opt = _options(grad_dtype, tau_max, delta_max, lr_at_server, params, device, select_mode,
                   compressor, seed, n_total, worker_base)
    ctx = _vp()
    _check(load().deco_init(ctypes.byref(ctx), d, n, delta, tau, lr, ctypes.byref(opt)),
           "deco_init")
    return ctx.value


def deco_layered_init(d, n, layer_offsets, delta, tau, lr, grad_dtype=DECO_F32, tau_max=0,
                      delta_max=0.0, lr_at_server=False, params=None, device=0,
                      select_mode=DECO_SELECT_AUTO, compressor=DECO_COMPRESSOR_TOPK, seed=0):
    """Per-layer Top-k: `layer_offsets` = [0, ..., d] (len = layers + 1).  -> opaque handle."""
    opt = _options(grad_dtype, tau_max, delta_max, lr_at_server, params, device, select_mode,
                   compressor, seed)
    offs = (_u64 * len(layer_offsets))(*[int(x) for x in layer_offsets])
    ctx = _vp()
    _check(load().deco_layered_init(ctypes.byref(ctx), d, n, offs, len(layer_offsets) - 1, delta,
                                    tau, lr, ctypes.byref(opt)), "deco_layered_init")
    return ctx.value


def deco_layered_destroy(ctx):
    load().deco_layered_destroy(ctx)


def deco_layered_step(ctx, grads, stream=None):
    _check(load().deco_layered_step(ctx, _ptr(grads), _stream(stream)), "deco_layered_step")


def deco_layered_join(ctx, stream=None):
    _check(load().deco_layered_join(ctx, _stream(stream)), "deco_layered_join")


def deco_layered_set_policy(ctx, delta, tau):
    _check(load().deco_layered_set_policy(ctx, delta, tau), "deco_layered_set_policy")


def deco_layered_set_lr(ctx, lr):
    _check(load().deco_layered_set_lr(ctx, lr), "deco_layered_set_lr")


def deco_layered_layer(ctx, layer):
    """-> (layer context handle, offset, length); the handle works with every deco_get_*."""
    c, off, ln = _vp(), _u64(), _u64()
    _check(load().deco_layered_layer(ctx, layer, ctypes.byref(c), ctypes.byref(off),
                                     ctypes.byref(ln)), "deco_layered_layer")
    return c.value, off.value, ln.value


def deco_layered_info(ctx):
    nl, kt, pp, st = _u32(), _u64(), _vp(), _u64()
    _check(load().deco_layered_info(ctx, ctypes.byref(nl), ctypes.byref(kt), ctypes.byref(pp),
                                    ctypes.byref(st)), "deco_layered_info")
    return {"n_layers": nl.value, "k_total": kt.value, "params": pp.value, "step": st.value}


def deco_destroy(ctx):
    load().deco_destroy(ctx)


def deco_reset(ctx, stream=None):
    _check(load().deco_reset(ctx, _stream(stream)), "deco_reset")


def deco_ef_compress(ctx, grads, stream=None):
    _check(load().deco_ef_compress(ctx, _ptr(grads), _stream(stream)), "deco_ef_compress")


def deco_aggregate_stale(ctx, stream=None):
    _check(load().deco_aggregate_stale(ctx, _stream(stream)), "deco_aggregate_stale")


def deco_apply_update(ctx, stream=None):
    _check(load().deco_apply_update(ctx, _stream(stream)), "deco_apply_update")


def deco_step(ctx, grads, stream=None):
    _check(load().deco_step(ctx, _ptr(grads), _stream(stream)), "deco_step")


def deco_join(ctx, stream=None):
    _check(load().deco_join(ctx, _stream(stream)), "deco_join")


def deco_step_host(ctx, grads_host, msg_host_out=None, params_host_out=None, stream=None):
    _check(load().deco_step_host(ctx, _ptr(grads_host), _ptr(msg_host_out),
                                 _ptr(params_host_out), _stream(stream)), "deco_step_host")


def deco_set_policy(ctx, delta, tau):
    _check(load().deco_set_policy(ctx, delta, tau), "deco_set_policy")


def deco_set_lr(ctx, lr):
    _check(load().deco_set_lr(ctx, lr), "deco_set_lr")


def deco_policy_select(V_g_bits, a_bar_bps, b_s, T_comp_s, tau_cap=0, non_iid=False):
    """Algorithm 3 -> (tau, delta)."""
    tau, delta = _u32(), _f64()
    _check(load().deco_policy_select(V_g_bits, a_bar_bps, b_s, T_comp_s, tau_cap,
                                     int(bool(non_iid)), ctypes.byref(tau),
                                     ctypes.byref(delta)), "deco_policy_select")
    return tau.value, delta.value


def deco_lut_build(V_g_bits, a_min_bps, a_max_bps, b_s, T_comp_s, points=20, tau_cap=0,
                   non_iid=False):
    """-> ctypes array of `points` deco_lut_entry (bandwidth sample, delta, tau)."""
    lut = (deco_lut_entry * points)()
    _check(load().deco_lut_build(V_g_bits, a_min_bps, a_max_bps, b_s, T_comp_s, points, tau_cap,
                                 int(bool(non_iid)), lut), "deco_lut_build")
    return lut


def deco_lut_lookup(lut, a_bar_bps, V_g_bits, b_s, T_comp_s, tau_cap=0, non_iid=False):
    """Nearest sample inside the profiled range, online DeCo outside -> (tau, delta)."""
    tau, delta = _u32(), _f64()
    _check(load().deco_lut_lookup(lut, len(lut), a_bar_bps, V_g_bits, b_s, T_comp_s, tau_cap,
                                  int(bool(non_iid)), ctypes.byref(tau), ctypes.byref(delta)),
           "deco_lut_lookup")
    return tau.value, delta.value


def deco_t_avg(delta, tau, V_g_bits, a_bar_bps, b_s, T_comp_s):
    return load().deco_t_avg(delta, tau, V_g_bits, a_bar_bps, b_s, T_comp_s)


def deco_k_from_delta(delta, d):
    return load().deco_k_from_delta(delta, d)


def deco_get_k(ctx):
    k = _u64()
    _check(load().deco_get_k(ctx, ctypes.byref(k)), "deco_get_k")
    return k.value


def deco_get_buffers(ctx):
    """-> dict of raw device addresses and sizes: e, e_stride, msg, k_cap, params."""
    e, msg, params = _vp(), _vp(), _vp()
    stride, k_cap = _u64(), _u64()
    _check(load().deco_get_buffers(ctx, ctypes.byref(e), ctypes.byref(stride), ctypes.byref(msg),
                                   ctypes.byref(k_cap), ctypes.byref(params)),
           "deco_get_buffers")
    return {"e": e.value, "e_stride": stride.value, "msg": msg.value, "k_cap": k_cap.value,
            "params": params.value}


def deco_get_aggregate(ctx, step):
    """-> (device address of the pairs, number of positions) of a cached aggregate."""
    entries, positions = _vp(), _u64()
    _check(load().deco_get_aggregate(ctx, step, ctypes.byref(entries), ctypes.byref(positions)),
           "deco_get_aggregate")
    return entries.value, positions.value


def deco_get_aggregate_vector(ctx, step):
    """-> device address of the d fp32 values of a cached aggregate kept as a plain vector."""
    values = _vp()
    _check(load().deco_get_aggregate_vector(ctx, step, ctypes.byref(values)),
           "deco_get_aggregate_vector")
    return values.value


def deco_get_select_info(ctx, n, stream=None):
    """-> (threshold_key[n], n_greater[n], exact_passes[n]) as Python lists."""
    thr, gt, ex = (_u32 * n)(), (_u32 * n)(), (_u32 * n)()
    _check(load().deco_get_select_info(ctx, _stream(stream), thr, gt, ex),
           "deco_get_select_info")
    return list(thr), list(gt), list(ex)


def deco_get_stats(ctx, stream=None):
    st = deco_stats()
    _check(load().deco_get_stats(ctx, _stream(stream), ctypes.byref(st)), "deco_get_stats")
    return {f: getattr(st, f) for f, _ in deco_stats._fields_}


def deco_set_kernel_timing(ctx, enabled):
    _check(load().deco_set_kernel_timing(ctx, int(bool(enabled))), "deco_set_kernel_timing")


def deco_get_kernel_timing(ctx, stream=None):
    """-> ({'accumulate','select','aggregate','apply'}: summed ms, iterations covered)."""
    ms = (_f64 * 4)()
    it = _u64()
    _check(load().deco_get_kernel_timing(ctx, _stream(stream), ms, ctypes.byref(it)),
           "deco_get_kernel_timing")
    return dict(zip(("accumulate", "select", "aggregate", "apply"), list(ms))), it.value


def deco_state_bytes(ctx):
    n = _u64()
    _check(load().deco_state_bytes(ctx, ctypes.byref(n)), "deco_state_bytes")
    return n.value


def deco_export_state(ctx, stream=None):
    """-> bytes object holding the checkpoint of the context."""
    n = deco_state_bytes(ctx)
    buf = ctypes.create_string_buffer(n)
    _check(load().deco_export_state(ctx, buf, n, _stream(stream)), "deco_export_state")
    return buf.raw


def deco_import_state(ctx, blob, stream=None):
    _check(load().deco_import_state(ctx, blob, len(blob), _stream(stream)), "deco_import_state")


def deco_launch_count(ctx):
    return load().deco_launch_count(ctx)


def deco_get_exchange(ctx):
    """The exchange buffer of a worker-sharded context: what the job all-gathers between
    compress and aggregate."""
    rows, rw = _vp(), _u64()
    r0, rl, rt = _u32(), _u32(), _u32()
    _check(load().deco_get_exchange(ctx, ctypes.byref(rows), ctypes.byref(rw), ctypes.byref(r0),
                                    ctypes.byref(rl), ctypes.byref(rt)), "deco_get_exchange")
    return {"rows": rows.value, "row_words": rw.value, "row0": r0.value, "rows_local": rl.value,
            "rows_total": rt.value}


def exchange_view(ctx, device=0):
    """torch view [rows_total, row_words] int32 of the exchange buffer at the current k (rows
    back to back: contiguous), for one torch.distributed collective or plain copies."""
    x = deco_get_exchange(ctx)
    return view_i32(x["rows"], (x["rows_total"], x["row_words"]), device), x


def all_gather_rows(full, row0, rows_local, group=None):
    """In-place all-gather of a row-sharded contiguous tensor: this rank owns rows
    [row0, row0 + rows_local) of `full`, every rank the same number, in rank order.  One
    collective.  Plumbing (torch.distributed)."""
    import torch.distributed as dist
    mine = full[row0:row0 + rows_local]
    dist.all_gather_into_tensor(full, mine, group=group)


def deco_step_sharded(ctx, grads, group=None, stream=None, device=0):
    """One iteration of a worker-sharded context: compress the local workers, all-gather the
    exchange rows (k pairs and the tile directory of every worker) among the ranks of `group`
    with one collective (NCCL on GPUs: it runs on torch's current stream, which must be
    `stream`), aggregate, update."""
    deco_ef_compress(ctx, grads, stream)
    rows, x = exchange_view(ctx, device)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        all_gather_rows(rows, x["row0"], x["rows_local"], group)
    elif x["rows_total"] != x["rows_local"]:
        raise RuntimeError("a worker-sharded context needs an initialised process group")
    deco_aggregate_stale(ctx, stream)
    deco_apply_update(ctx, stream)


DECO_STATIC_MAX_D = 16777216


def deco_topk_compress_static(a, d, k, msg_out, stream=None):
    """Top-k of one fp32 CUDA tensor `a` into `msg_out` ([k, 2] int32 view of the pairs), with
    no allocation inside the library (fixed device scratch; d <= DECO_STATIC_MAX_D).  For
    callers that cannot allocate: during stream capture, under a foreign memory pool."""
    _check(load().deco_topk_compress_static(_ptr(a), d, k, _ptr(msg_out), _stream(stream)),
           "deco_topk_compress_static")


# ------------------------------------------------------------- device views (plumbing)

class _DevArray:
    """Minimal __cuda_array_interface__ holder so torch can view library-owned memory."""

    def __init__(self, addr, shape, typestr, strides=None):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr,
                                         "data": (int(addr), False), "version": 2,
                                         "strides": strides}


def view_f32(addr, shape, device=0):
    import torch
    return torch.as_tensor(_DevArray(addr, shape, "<f4"), device="cuda:%d" % device)


def view_i32(addr, shape, device=0):
    import torch
    return torch.as_tensor(_DevArray(addr, shape, "<i4"), device="cuda:%d" % device)
