"""CPU oracle for one round of double quantization -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy binding over ``dq_oracle.c`` (plain C, compiled with
``-O2 -ffp-contract=off``).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library never
does, and the two share no code.  Every function here forwards to the C
function of the same name (``dqo_`` prefix dropped); the C file cites the
passage of the paper each one follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dq_oracle.c")
_LIB = os.path.join(_HERE, "libdq_oracle.so")

DENSE_F32, CSR_F32, DENSE_BF16 = 0, 1, 2
MSG_DENSE, MSG_SPARSE = 0, 1
STREAM_MODEL, STREAM_GRAD, STREAM_MASK, STREAM_BATCH = 0, 1, 2, 3
MASTER = 0xFFFFFFFF
OK, ERR_ARG, ERR_NONFINITE = 0, 1, 4


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


class Data(C.Structure):
    _fields_ = [("format", C.c_int32), ("pad_", C.c_int32), ("n", C.c_int64), ("d", C.c_int64),
                ("values", C.c_void_p), ("col_idx", C.c_void_p), ("row_ptr", C.c_void_p), ("labels", C.c_void_p)]


class Config(C.Structure):
    _fields_ = [("d", C.c_int64), ("M", C.c_int32), ("B", C.c_int32), ("bx", C.c_int32), ("b", C.c_int32),
                ("l1", C.c_float), ("l2", C.c_float), ("box_lo", C.c_float), ("box_hi", C.c_float),
                ("sparsify", C.c_int32), ("phi", C.c_float),
                ("msg_format", C.c_int32), ("accelerated", C.c_int32), ("snapshot_flag", C.c_int32), ("pad_", C.c_int32),
                ("seed", C.c_uint64), ("mu", C.c_float), ("sequential", C.c_int32),
                ("model", C.c_int32), ("hidden", C.c_int32), ("classes", C.c_int32), ("pad3_", C.c_int32)]


class State(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("x", "xsnap", "gfull", "y", "xsum")]


class Trace(C.Structure):
    _fields_ = [("codes_x", C.c_void_p), ("delta_x", C.c_void_p), ("xhat", C.c_void_p), ("rows", C.c_void_p),
                ("alpha", C.c_void_p), ("S", C.c_void_p), ("beta", C.c_void_p), ("Z", C.c_void_p),
                ("codes", C.c_void_p), ("delta", C.c_void_p), ("ninf", C.c_void_p), ("n1", C.c_void_p),
                ("phi_eff", C.c_void_p), ("nnz", C.c_void_p),
                ("bits_down", C.c_uint64), ("bits_up", C.c_uint64), ("normx", C.c_float), ("flag_round", C.c_int32),
                ("bx_used", C.c_int32), ("pad_", C.c_int32)]


def _declare(L):
    u32, u64, i32, i64, f32, f64, vp = C.c_uint32, C.c_uint64, C.c_int32, C.c_int64, C.c_float, C.c_double, C.c_void_p
    sig = {
        "dqo_philox4x32_10": (None, [vp, vp, vp]),
        "dqo_u16": (u32, [u64, u32, u32, u32, u64]),
        "dqo_u15": (u32, [u64, u32, u32, u32, u64]),
        "dqo_scale_delta": (f32, [f32, i32]),
        "dqo_scale_inv": (f32, [f32, i32]),
        "dqo_q_code": (i32, [f32, f32, i32, u32]),
        "dqo_norm_inf": (f32, [vp, i64]),
        "dqo_norm_l1": (f32, [vp, i64, f32]),
        "dqo_quantize": (i32, [vp, i64, i32, u64, u32, u32, u32, vp, vp]),
        "dqo_pack": (None, [vp, i64, i32, vp, i64]),
        "dqo_unpack": (None, [vp, i64, i32, vp]),
        "dqo_sparsify": (i32, [vp, i64, f32, u64, u32, u32, vp, vp, vp, vp, vp, vp]),
        "dqo_quantize_survivors": (i32, [vp, vp, i64, i32, u64, u32, u32, vp, vp]),
        "dqo_margin": (f64, [vp, i64, vp]),
        "dqo_worker_grad": (None, [vp, vp, vp, vp, i32, vp, vp]),
        "dqo_full_grad": (None, [vp, vp, vp, vp]),
        "dqo_smooth_loss": (f64, [vp, vp]),
        "dqo_objective": (f64, [vp, vp, f32, f32]),
        "dqo_sample_batch": (None, [u64, u32, i32, i32, i64, i32, vp]),
        "dqo_prox": (f32, [f32, f32, f32, f32, f32, f32]),
        "dqo_master_step": (None, [vp, vp, i32, i64, vp, vp, vp, vp, vp, f32, f32, i32, f32, f32, f32, f32, vp]),
        "dqo_epoch_begin": (None, [vp, vp, vp, f32, i64, vp]),
        "dqo_mlp_params": (i64, [i64, i32, i32]),
        "dqo_mlp_loss": (f64, [vp, i32, i32, vp, vp, i64]),
        "dqo_mlp_grad": (None, [vp, i32, i32, vp, vp, i64, vp]),
        "dqo_mlp_worker_grad": (None, [vp, i32, i32, vp, vp, vp, i32, vp, vp]),
        "dqo_mlp_objective": (f64, [vp, i32, i32, vp, f32, f32]),
        "dqo_master_step_sequential": (None, [vp, vp, i32, i64, vp, vp, vp, vp, vp, f32, f32, i32, f32, f32, f32, f32, vp]),
        "dqo_expected_sq_error": (f64, [vp, i64, i32]),
        "dqo_sq_distance": (f64, [vp, vp, i64]),
        "dqo_select_bx": (i32, [vp, vp, i64, f32, vp, vp]),
        "dqo_round": (i32, [vp, vp, vp, u32, i32, f32, f32, vp]),
        "dqo_round_delayed": (i32, [vp, vp, vp, u32, i32, f32, f32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args


def _p(a):
    return None if a is None else a.ctypes.data


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ---- RNG --------------------------------------------------------------------
def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32); k = np.asarray(key, dtype=np.uint32); o = np.zeros(4, np.uint32)
    lib().dqo_philox4x32_10(_p(c), _p(k), _p(o))
    return o


def u16(seed, round_, worker, stream, i):
    return int(lib().dqo_u16(seed, round_, worker, stream, i))


def u15(seed, round_, worker, stream, i):
    return int(lib().dqo_u15(seed, round_, worker, stream, i))


# ---- quantiser ----------------------------------------------------------------
def scale_delta(nrm, b):
    return np.float32(lib().dqo_scale_delta(float(nrm), b))


def scale_inv(nrm, b):
    return np.float32(lib().dqo_scale_inv(float(nrm), b))


def q_code(v, inv, b, u15_):
    return int(lib().dqo_q_code(float(v), float(inv), b, u15_))


def norm_inf(v):
    v = _f32(v)
    return np.float32(lib().dqo_norm_inf(_p(v), v.size))


def norm_l1(v, ninf=None):
    v = _f32(v)
    if ninf is None:
        ninf = norm_inf(v)
    return np.float32(lib().dqo_norm_l1(_p(v), v.size, float(ninf)))


def quantize(v, b, seed, round_, worker, stream):
    """Q_(delta,b)(v) with delta = ||v||_inf/(2^(b-1)-1): returns (codes int32[d], delta, status)."""
    v = _f32(v)
    codes = np.zeros(v.size, np.int32); delta = np.zeros(1, np.float32)
    rc = lib().dqo_quantize(_p(v), v.size, b, seed, round_, worker, stream, _p(codes), _p(delta))
    return codes, delta[0], rc


def pack(codes, b, out_bytes=None):
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    nb = (codes.size * b + 7) // 8
    if out_bytes is None:
        out_bytes = (nb + 15) // 16 * 16
    out = np.zeros(out_bytes, np.uint8)
    lib().dqo_pack(_p(codes), codes.size, b, _p(out), out.size)
    return out


def unpack(buf, count, b):
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    codes = np.zeros(count, np.int32)
    lib().dqo_unpack(_p(buf), count, b, _p(codes))
    return codes


# ---- sparsifier -----------------------------------------------------------------
def sparsify(alpha, phi, seed, round_, worker):
    """eq. (4): returns dict(beta, Z, m (p_i*2^16), ninf, n1, phi_eff, status)."""
    alpha = _f32(alpha); d = alpha.size
    beta = np.zeros(d, np.float32); Z = np.zeros(d, np.uint8); m = np.zeros(d, np.uint32)
    s = np.zeros(3, np.float32)
    rc = lib().dqo_sparsify(_p(alpha), d, float(phi), seed, round_, worker, _p(beta), _p(Z), _p(m),
                            s[0:1].ctypes.data, s[1:2].ctypes.data, s[2:3].ctypes.data)
    return dict(beta=beta, Z=Z, m=m, ninf=s[0], n1=s[1], phi_eff=s[2], status=rc)


def quantize_survivors(beta, Z, b, seed, round_, worker):
    beta = _f32(beta); Z = np.ascontiguousarray(Z, dtype=np.uint8)
    codes = np.zeros(beta.size, np.int32); delta = np.zeros(1, np.float32)
    rc = lib().dqo_quantize_survivors(_p(beta), _p(Z), beta.size, b, seed, round_, worker, _p(codes), _p(delta))
    return codes, delta[0], rc


# ---- data + gradients -------------------------------------------------------------
class Dataset:
    """Host copy of the training matrix in one of the three formats the library takes."""

    def __init__(self, fmt, n, d, values, labels, col_idx=None, row_ptr=None):
        self.format, self.n, self.d = fmt, int(n), int(d)
        if fmt == DENSE_BF16:
            self.values = np.ascontiguousarray(values, dtype=np.uint16)      # raw bf16 bit patterns
        else:
            self.values = np.ascontiguousarray(values, dtype=np.float32)
        self.labels = np.ascontiguousarray(labels, dtype=np.float32)
        self.col_idx = None if col_idx is None else np.ascontiguousarray(col_idx, dtype=np.int32)
        self.row_ptr = None if row_ptr is None else np.ascontiguousarray(row_ptr, dtype=np.int64)
        self.c = Data(fmt, 0, self.n, self.d, _p(self.values), _p(self.col_idx), _p(self.row_ptr), _p(self.labels))

    @property
    def ref(self):
        return C.addressof(self.c)


def margin(data, row, x):
    x = _f32(x)
    return float(lib().dqo_margin(data.ref, row, _p(x)))


def worker_grad(data, xhat, xsnap, rows):
    xhat, xsnap = _f32(xhat), _f32(xsnap)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    alpha = np.zeros(data.d, np.float32); S = np.zeros(data.d, np.float32)
    lib().dqo_worker_grad(data.ref, _p(xhat), _p(xsnap), _p(rows), rows.size, _p(alpha), _p(S))
    return alpha, S


def full_grad(data, x):
    x = _f32(x)
    g = np.zeros(data.d, np.float32); z = np.zeros(data.n, np.float32)
    lib().dqo_full_grad(data.ref, _p(x), _p(g), _p(z))
    return g, z


def smooth_loss(data, x):
    x = _f32(x)
    return float(lib().dqo_smooth_loss(data.ref, _p(x)))


def objective(data, x, l1, l2):
    x = _f32(x)
    return float(lib().dqo_objective(data.ref, _p(x), float(l1), float(l2)))


def sample_batch(seed, round_, w, M, n, B):
    rows = np.zeros(B, np.int64)
    lib().dqo_sample_batch(seed, round_, w, M, n, B, _p(rows))
    return rows


# ---- the 3-layer network --------------------------------------------------------------------------------
MODEL_LOGISTIC, MODEL_MLP = 0, 1


def mlp_params(n_in, hidden, classes):
    return int(lib().dqo_mlp_params(n_in, hidden, classes))


def mlp_loss(data, hidden, classes, x, rows=None):
    x = _f32(x)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    return float(lib().dqo_mlp_loss(data.ref, hidden, classes, _p(x), _p(r), data.n if r is None else r.size))


def mlp_grad(data, hidden, classes, x, rows=None):
    x = _f32(x)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    g = np.zeros(mlp_params(data.d, hidden, classes), np.float32)
    lib().dqo_mlp_grad(data.ref, hidden, classes, _p(x), _p(r), data.n if r is None else r.size, _p(g))
    return g


def mlp_worker_grad(data, hidden, classes, xhat, xsnap, rows):
    xhat, xsnap = _f32(xhat), _f32(xsnap)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    P = mlp_params(data.d, hidden, classes)
    alpha = np.zeros(P, np.float32); S = np.zeros(P, np.float32)
    lib().dqo_mlp_worker_grad(data.ref, hidden, classes, _p(xhat), _p(xsnap), _p(rows), rows.size, _p(alpha), _p(S))
    return alpha, S


def mlp_objective(data, hidden, classes, x, l1, l2):
    x = _f32(x)
    return float(lib().dqo_mlp_objective(data.ref, hidden, classes, _p(x), float(l1), float(l2)))


# ---- master -----------------------------------------------------------------------
def prox(v, eta, l1, l2, lo, hi):
    return np.float32(lib().dqo_prox(float(v), float(eta), float(l1), float(l2), float(lo), float(hi)))


def master_step(codes, delta, gfull, x, eta, theta=0.0, accelerated=False, y=None, xsnap=None, xsum=None,
                l1=0.0, l2=0.0, lo=-np.inf, hi=np.inf, sequential=False):
    """Updates x (and y, xsum) in place; returns ||x||_inf.  sequential: one prox step per message."""
    codes = np.ascontiguousarray(codes, dtype=np.int32); M, d = codes.shape
    delta = _f32(delta); gfull = _f32(gfull)
    for a in (x, y, xsum):
        assert a is None or (a.dtype == np.float32 and a.flags.c_contiguous)
    xsnap_ = None if xsnap is None else _f32(xsnap)
    nx = np.zeros(1, np.float32)
    fn = lib().dqo_master_step_sequential if sequential else lib().dqo_master_step
    fn(_p(codes), _p(delta), M, d, _p(gfull), _p(x), _p(y), _p(xsnap_), _p(xsum),
                          float(eta), float(theta), int(accelerated), float(l1), float(l2), float(lo), float(hi), _p(nx))
    return nx[0]


# ---- model precision (condition (3)) ----------------------------------------------------------------
def expected_sq_error(x, b):
    x = _f32(x)
    return float(lib().dqo_expected_sq_error(_p(x), x.size, b))


def select_bx(x, xsnap, mu):
    """Returns (chosen width, expected errors at 2..11 bits, ||x - xsnap||^2)."""
    x, xsnap = _f32(x), _f32(xsnap)
    err = np.zeros(10, np.float64); dist = np.zeros(1, np.float64)
    b = lib().dqo_select_bx(_p(x), _p(xsnap), x.size, float(mu), _p(err), _p(dist))
    return int(b), err, float(dist[0])


# ---- drivers ------------------------------------------------------------------------
def make_config(d, M, B, bx, b, l1=0.0, l2=0.0, box_lo=-np.inf, box_hi=np.inf, sparsify=0, phi=0.0,
                msg_format=MSG_DENSE, accelerated=0, snapshot_flag=1, seed=0, mu=0.0, sequential=0, model=0, hidden=0, classes=0):
    return Config(d, M, B, bx, b, l1, l2, box_lo, box_hi, int(sparsify), phi, msg_format, int(accelerated),
                  int(snapshot_flag), 0, seed, mu, int(sequential), int(model), int(hidden), int(classes), 0)


class Run:
    """State of one optimisation run (x, snapshot, full gradient, and y / xsum for Algorithm 3)."""

    def __init__(self, cfg: Config, data: Dataset, x0):
        self.cfg, self.data = cfg, data
        d = cfg.d
        self.x = _f32(x0).copy(); self.xsnap = self.x.copy(); self.gfull = np.zeros(d, np.float32)
        self.y = self.x.copy(); self.xsum = np.zeros(d, np.float32)
        self.z_snap = np.zeros(data.n, np.float32)
        self.state = State(_p(self.x), _p(self.xsnap), _p(self.gfull), _p(self.y), _p(self.xsum))
        self.rounds_in_epoch = 0
        self.ticks_in_epoch = 0
        self.epoch = -1

    def epoch_begin(self, theta=0.0):
        lib().dqo_epoch_begin(C.addressof(self.cfg), self.data.ref, C.addressof(self.state), float(theta),
                              self.ticks_in_epoch, _p(self.z_snap))       # Algorithm 3 averages over master ticks
        self.rounds_in_epoch = 0
        self.ticks_in_epoch = 0
        self.epoch += 1

    def is_flag_round(self):
        """The model equals the snapshot at the first round of an epoch of Algorithms 1/2, and of the
        first epoch of Algorithm 3 (where y_0 = xsnap makes x_0 = xsnap)."""
        if not self.cfg.snapshot_flag or self.rounds_in_epoch != 0:
            return False
        return (not self.cfg.accelerated) or self.epoch == 0

    def round(self, round_, eta, theta=0.0, trace=False, delays=None, across_epochs=False):
        """delays: per worker, how many rounds ago the model it works on was broadcast (Algorithm 1's t - D(t)).  By
        default a delay is cut to the rounds the epoch has had; with across_epochs it may reach back into the
        previous epoch (cut to the rounds the run has had): the worker then evaluates the previous epoch's
        low-precision model against THIS epoch's snapshot and full gradient, as step 11 is written.  The run keeps
        the broadcasts for that."""
        cfg = self.cfg; d, M, B = cfg.d, cfg.M, cfg.B
        flag = self.is_flag_round()
        T = Trace(); keep = {}
        if delays is not None and not trace:
            keep = dict(xhat=np.zeros(d, np.float32)); T.xhat = _p(keep["xhat"])
        if trace:
            keep = dict(codes_x=np.zeros(d, np.int32), delta_x=np.zeros(1, np.float32), xhat=np.zeros(d, np.float32),
                        rows=np.zeros((M, B), np.int64), alpha=np.zeros((M, d), np.float32),
                        S=np.zeros((M, d), np.float32), beta=np.zeros((M, d), np.float32),
                        Z=np.zeros((M, d), np.uint8), codes=np.zeros((M, d), np.int32),
                        delta=np.zeros(M, np.float32), ninf=np.zeros(M, np.float32), n1=np.zeros(M, np.float32),
                        phi_eff=np.zeros(M, np.float32), nnz=np.zeros(M, np.int64))
            for k, a in keep.items():
                setattr(T, k, _p(a))
        if delays is None:
            rc = lib().dqo_round(C.addressof(cfg), self.data.ref, C.addressof(self.state), round_, int(flag),
                                 float(eta), float(theta), C.addressof(T))
        else:
            if not hasattr(self, "broadcasts") or (self.rounds_in_epoch == 0 and not across_epochs):
                self.broadcasts = []                                       # low-precision models by round (of this epoch, or of the run)
            t = len(self.broadcasts)
            used = [min(int(D), t) for D in delays]
            ptrs = (C.c_void_p * M)(*[None if D == 0 else _p(self.broadcasts[t - D]) for D in used])
            rc = lib().dqo_round_delayed(C.addressof(cfg), self.data.ref, C.addressof(self.state), round_, int(flag),
                                         float(eta), float(theta), C.addressof(T), ptrs)
            self.broadcasts.append(keep["xhat"].copy())
            keep["delays_used"] = used
        self.rounds_in_epoch += 1
        self.ticks_in_epoch += cfg.M if cfg.sequential else 1
        keep.update(bits_down=int(T.bits_down), bits_up=int(T.bits_up), normx=np.float32(T.normx),
                    flag_round=bool(T.flag_round), bx_used=int(T.bx_used), status=rc)
        return keep
