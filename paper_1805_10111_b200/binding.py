"""ctypes binding of libdq.so: the same entry points as include/dq.h, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams are torch's); every step of the round runs in
the library's kernels.  Importing this module does not need a GPU; calling into it does.  If libdq.so has
not been built the first call raises -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdq.so")

DQ_OK, DQ_ERR_ARG, DQ_ERR_SHAPE, DQ_ERR_BITS, DQ_ERR_NONFINITE, DQ_ERR_CAPACITY, DQ_ERR_CUDA, DQ_ERR_TIMEOUT = range(8)
DQ_DENSE_F32, DQ_CSR_F32, DQ_DENSE_BF16 = 0, 1, 2
DQ_MSG_DENSE, DQ_MSG_SPARSE = 0, 1
DQ_MODEL_LOGISTIC, DQ_MODEL_MLP = 0, 1

EXPORTS = ["dq_packed_bytes", "dq_create", "dq_destroy", "dq_epoch_begin", "dq_quantize_model", "dq_worker_grad",
           "dq_norm_inf", "dq_quantize_sparsify_pack", "dq_master_unpack_aggregate_prox", "dq_round", "dq_codec_round",
           "dq_codec_host_setup", "dq_codec_round_host", "dq_unpack", "dq_objective", "dq_round_buffers",
           "dq_poll_status", "dq_launch_count", "dq_strerror", "dq_quantize_pack_static", "dq_select_model_bits",
           "dq_last_model_bits", "dq_rounds", "dq_set_delays"]


class dq_data(C.Structure):
    _fields_ = [("format", C.c_int32), ("reserved", C.c_int32), ("n", C.c_int64), ("d", C.c_int64),
                ("values", C.c_void_p), ("col_idx", C.c_void_p), ("row_ptr", C.c_void_p), ("labels", C.c_void_p)]


class dq_config(C.Structure):
    _fields_ = [("d", C.c_int64), ("M", C.c_int32), ("B", C.c_int32), ("bx", C.c_int32), ("b", C.c_int32),
                ("lambda1", C.c_float), ("lambda2", C.c_float), ("box_lo", C.c_float), ("box_hi", C.c_float),
                ("sparsify", C.c_int32), ("phi", C.c_float), ("msg_format", C.c_int32), ("accelerated", C.c_int32),
                ("snapshot_flag", C.c_int32), ("no_graph", C.c_int32), ("seed", C.c_uint64), ("sparse_cap", C.c_int64), ("mu", C.c_float), ("sequential", C.c_int32),
                ("model", C.c_int32), ("hidden", C.c_int32), ("classes", C.c_int32), ("no_fused", C.c_int32), ("max_delay", C.c_int32),
                ("tensor_cores", C.c_int32), ("delay_across_epochs", C.c_int32)]


class dq_state(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("x", "x_snap", "g_full", "y", "x_sum", "norm_x", "z_snap")]


class dq_msgs(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("stride", C.c_int64), ("scale", C.c_void_p),
                ("idx", C.c_void_p), ("cap", C.c_int64), ("nnz", C.c_void_p)]


class DqError(RuntimeError):
    def __init__(self, status, where=""):
        self.status = status
        super().__init__("%s: status %d (%s)" % (where or "libdq", status, dq_strerror(status)))


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built (python -m paper_1805_10111_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libdq.so is missing at %s: build it with `python -m paper_1805_10111_b200.build`; "
                               "there is no fallback implementation" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u32, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_float
        sig = {
            "dq_packed_bytes": (i64, [i64, i32]),
            "dq_create": (i32, [C.POINTER(vp), C.POINTER(dq_config), C.POINTER(dq_data)]),
            "dq_destroy": (i32, [vp]),
            "dq_epoch_begin": (i32, [vp, C.POINTER(dq_state), f32, vp]),
            "dq_quantize_model": (i32, [vp, vp, vp, u32, vp, vp, vp]),
            "dq_worker_grad": (i32, [vp, vp, vp, i32, C.POINTER(dq_state), u32, vp, vp, vp, vp]),
            "dq_norm_inf": (i32, [vp, vp, i32, vp, vp]),
            "dq_quantize_sparsify_pack": (i32, [vp, vp, vp, u32, C.POINTER(dq_msgs), vp]),
            "dq_master_unpack_aggregate_prox": (i32, [vp, C.POINTER(dq_msgs), C.POINTER(dq_state), f32, f32, vp]),
            "dq_round": (i32, [vp, C.POINTER(dq_state), u32, f32, f32, vp, vp, vp]),
            "dq_rounds": (i32, [vp, C.POINTER(dq_state), u32, i32, f32, f32, vp, vp, vp]),
            "dq_set_delays": (i32, [vp, vp]),
            "dq_codec_round": (i32, [vp, vp, C.POINTER(dq_state), u32, f32, f32, vp, vp, vp]),
            "dq_codec_host_setup": (i32, [vp, vp, vp]),
            "dq_codec_round_host": (i32, [vp, vp, u32, f32, vp, vp, vp]),
            "dq_unpack": (i32, [vp, C.POINTER(dq_msgs), i32, vp, vp]),
            "dq_objective": (i32, [vp, vp, vp, vp]),
            "dq_round_buffers": (i32, [vp, C.POINTER(dq_msgs), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]),
            "dq_poll_status": (i32, [vp, C.POINTER(C.c_int), vp]),
            "dq_launch_count": (i64, [vp]),
            "dq_strerror": (C.c_char_p, [i32]),
            "dq_select_model_bits": (i32, [vp, vp, vp, vp, f32, vp, vp, vp]),
            "dq_last_model_bits": (i32, [vp, C.POINTER(C.c_int32), vp]),
            "dq_quantize_pack_static": (i32, [vp, i64, i32, i32, C.c_uint64, u32, vp, i64, vp, vp]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t):
    """Device (or host) address of a tensor / numpy array / None."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream):
    if stream is not None:
        return stream
    import torch
    return torch.cuda.current_stream().cuda_stream


# ---- holders that keep the tensors behind the C structs alive ------------------------------------------------
class Data:
    """Device copy of a training set (see synth.HostData) and its dq_data view."""

    def __init__(self, host, device="cuda"):
        import torch
        self.format, self.n, self.d = host.format, host.n, host.d
        if host.format == DQ_DENSE_BF16:
            self.values = torch.from_numpy(host.values.view("int16")).to(device).view(torch.bfloat16)
        else:
            self.values = torch.from_numpy(host.values).to(device)
        self.labels = torch.from_numpy(host.labels).to(device)
        self.col_idx = None if host.col_idx is None else torch.from_numpy(host.col_idx).to(device)
        self.row_ptr = None if host.row_ptr is None else torch.from_numpy(host.row_ptr).to(device)
        self.c = dq_data(host.format, 0, host.n, host.d, _ptr(self.values), _ptr(self.col_idx), _ptr(self.row_ptr),
                         _ptr(self.labels))


class State:
    """Optimiser state tensors on the device and their dq_state view."""

    def __init__(self, x0, n=0, accelerated=False, device="cuda"):
        import torch
        self.x = torch.as_tensor(x0, dtype=torch.float32).to(device).contiguous().clone()
        d = self.x.numel()
        self.x_snap = self.x.clone()
        self.g_full = torch.zeros(d, dtype=torch.float32, device=device)
        self.y = self.x.clone() if accelerated else None
        self.x_sum = torch.zeros(d, dtype=torch.float32, device=device) if accelerated else None
        self.norm_x = torch.zeros(1, dtype=torch.float32, device=device)
        self.z_snap = torch.zeros(max(n, 1), dtype=torch.float32, device=device)
        self.c = dq_state(_ptr(self.x), _ptr(self.x_snap), _ptr(self.g_full), _ptr(self.y), _ptr(self.x_sum),
                          _ptr(self.norm_x), _ptr(self.z_snap))


class Msgs:
    """Buffers for M worker messages and their dq_msgs view."""

    def __init__(self, cfg: dq_config, cap=None, device="cuda"):
        import torch
        sparse = bool(cfg.sparsify) and cfg.msg_format == DQ_MSG_SPARSE
        self.cap = int(cap if cap is not None else cfg.d) if sparse else 0
        self.stride = int(dq_packed_bytes(self.cap if sparse else cfg.d, cfg.b))
        self.codes = torch.zeros((cfg.M, self.stride), dtype=torch.uint8, device=device)
        self.scale = torch.zeros(cfg.M, dtype=torch.float32, device=device)
        self.idx = torch.zeros((cfg.M, max(self.cap, 1)), dtype=torch.int32, device=device) if sparse else None
        self.nnz = torch.zeros(cfg.M, dtype=torch.int32, device=device) if sparse else None
        self.c = dq_msgs(_ptr(self.codes), self.stride, _ptr(self.scale), _ptr(self.idx), self.cap, _ptr(self.nnz))


def make_config(d, M, B=1, bx=8, b=8, lambda1=0.0, lambda2=0.0, box_lo=float("-inf"), box_hi=float("inf"), sparsify=0,
                phi=0.0, msg_format=DQ_MSG_DENSE, accelerated=0, snapshot_flag=1, seed=0, sparse_cap=0, no_graph=0, mu=0.0, sequential=0, model=0, hidden=0, classes=0, no_fused=0, max_delay=0, tensor_cores=0, delay_across_epochs=0) -> dq_config:
    return dq_config(d, M, B, bx, b, lambda1, lambda2, box_lo, box_hi, int(sparsify), phi, msg_format, int(accelerated),
                     int(snapshot_flag), int(no_graph), seed, sparse_cap, mu, int(sequential), int(model), int(hidden), int(classes), int(no_fused), int(max_delay), int(tensor_cores), int(delay_across_epochs))


# ---- entry points (same names and order of arguments as include/dq.h) ---------------------------------------------
def dq_packed_bytes(count, b):
    return int(lib().dq_packed_bytes(int(count), int(b)))


def dq_strerror(status):
    return lib().dq_strerror(int(status)).decode()


def dq_create(cfg: dq_config, data: Data | None = None):
    """Returns (status, ctx)."""
    ctx = C.c_void_p()
    rc = lib().dq_create(C.byref(ctx), C.byref(cfg), C.byref(data.c) if data is not None else None)
    return rc, (ctx if rc == DQ_OK else None)


def dq_destroy(ctx):
    return lib().dq_destroy(ctx)


def dq_epoch_begin(ctx, st: State, theta=0.0, stream=None):
    return lib().dq_epoch_begin(ctx, C.byref(st.c), float(theta), _stream(stream))


def dq_quantize_model(ctx, x, norm_x, round_, codes_x, delta_x, stream=None):
    return lib().dq_quantize_model(ctx, _ptr(x), _ptr(norm_x), int(round_), _ptr(codes_x), _ptr(delta_x), _stream(stream))


def dq_worker_grad(ctx, codes_x, delta_x, is_snapshot, st: State, round_, batch_idx, alpha, norm_inf, stream=None):
    return lib().dq_worker_grad(ctx, _ptr(codes_x), _ptr(delta_x), int(is_snapshot), C.byref(st.c), int(round_),
                                _ptr(batch_idx), _ptr(alpha), _ptr(norm_inf), _stream(stream))


def dq_norm_inf(ctx, v, M, norm_inf, stream=None):
    return lib().dq_norm_inf(ctx, _ptr(v), int(M), _ptr(norm_inf), _stream(stream))


def dq_quantize_sparsify_pack(ctx, v, norm_inf, round_, out: Msgs, stream=None):
    return lib().dq_quantize_sparsify_pack(ctx, _ptr(v), _ptr(norm_inf), int(round_), C.byref(out.c), _stream(stream))


def dq_master_unpack_aggregate_prox(ctx, msgs: Msgs, st: State, eta, theta=0.0, stream=None):
    return lib().dq_master_unpack_aggregate_prox(ctx, C.byref(msgs.c), C.byref(st.c), float(eta), float(theta), _stream(stream))


def dq_round(ctx, st: State, round_, eta, theta=0.0, bits_down=None, bits_up=None, stream=None):
    return lib().dq_round(ctx, C.byref(st.c), int(round_), float(eta), float(theta), _ptr(bits_down), _ptr(bits_up),
                          _stream(stream))


def dq_rounds(ctx, st: State, round0, nrounds, eta, theta=0.0, bits_down=None, bits_up=None, stream=None):
    return lib().dq_rounds(ctx, C.byref(st.c), int(round0), int(nrounds), float(eta), float(theta), _ptr(bits_down),
                           _ptr(bits_up), _stream(stream))


def dq_set_delays(ctx, delays):
    """delays: sequence of M ints (rounds each worker lags), or None for no delay."""
    if delays is None:
        return lib().dq_set_delays(ctx, None)
    arr = (C.c_int32 * len(delays))(*[int(v) for v in delays])
    return lib().dq_set_delays(ctx, C.cast(arr, C.c_void_p))


def dq_codec_round(ctx, v, st: State, round_, eta, theta, codes_x, delta_x, stream=None):
    return lib().dq_codec_round(ctx, _ptr(v), C.byref(st.c), int(round_), float(eta), float(theta), _ptr(codes_x),
                                _ptr(delta_x), _stream(stream))


def dq_codec_host_setup(ctx, x_host, g_full_host):
    return lib().dq_codec_host_setup(ctx, _ptr(x_host), _ptr(g_full_host))


def dq_codec_round_host(ctx, v_host, round_, eta, codes_x_host, delta_x_host, stream=None):
    return lib().dq_codec_round_host(ctx, _ptr(v_host), int(round_), float(eta), _ptr(codes_x_host), _ptr(delta_x_host),
                                     _stream(stream))


def dq_unpack(ctx, msgs: Msgs, w, out, stream=None):
    return lib().dq_unpack(ctx, C.byref(msgs.c), int(w), _ptr(out), _stream(stream))


def dq_objective(ctx, x, P, stream=None):
    return lib().dq_objective(ctx, _ptr(x), _ptr(P), _stream(stream))


def dq_round_buffers(ctx):
    """Returns (status, dict of raw device addresses and the dq_msgs view of the context's own buffers)."""
    m = dq_msgs()
    ptrs = [C.c_void_p() for _ in range(5)]
    rc = lib().dq_round_buffers(ctx, C.byref(m), *[C.byref(p) for p in ptrs])
    names = ("alpha", "norm_inf", "batch_idx", "codes_x", "delta_x")
    return rc, dict(msgs=m, **{k: p.value for k, p in zip(names, ptrs)})


def dq_poll_status(ctx, stream=None):
    """Returns (status of the call, sticky device status)."""
    s = C.c_int(0)
    rc = lib().dq_poll_status(ctx, C.byref(s), _stream(stream))
    return rc, s.value


def dq_launch_count(ctx):
    return int(lib().dq_launch_count(ctx))


def dq_select_model_bits(ctx, x, x_snap, norm_x, mu, bits, stats, stream=None):
    return lib().dq_select_model_bits(ctx, _ptr(x), _ptr(x_snap), _ptr(norm_x), float(mu), _ptr(bits), _ptr(stats), _stream(stream))


def dq_last_model_bits(ctx, stream=None):
    """Returns (status, width chosen by the last dq_round)."""
    v = C.c_int32(0)
    rc = lib().dq_last_model_bits(ctx, C.byref(v), _stream(stream))
    return rc, v.value


def dq_quantize_pack_static(v, d, M, b, seed, round_, codes, stride, scale, stream=None):
    """Context-free dense quantise + pack that allocates nothing (scratch is a fixed array inside the library)."""
    return lib().dq_quantize_pack_static(_ptr(v), int(d), int(M), int(b), int(seed), int(round_), _ptr(codes), int(stride),
                                         _ptr(scale), _stream(stream))


def ok(rc, where=""):
    if rc != DQ_OK:
        raise DqError(rc, where)


class _RawDevice:
    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = dict(shape=(int(count),), typestr=typestr, data=(int(ptr), False), version=2)


def device_view(ptr, count, dtype):
    """Zero-copy torch view of `count` elements of device memory at address `ptr` (owned by the library)."""
    import torch
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.uint8: "|u1"}[dtype]
    return torch.as_tensor(_RawDevice(ptr, count, typestr), device="cuda")
