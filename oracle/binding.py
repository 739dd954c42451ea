"""ctypes access to the C++ oracle (``laq_oracle.cpp``) -- test infrastructure only.

The shared object is compiled on first use with
``g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math`` so that no operation is fused or
reordered.  Nothing here does arithmetic of the method: it only marshals numpy arrays.
"""
import ctypes as C
import os
import subprocess
import numpy as np

MODEL_LOGREG_BIN, MODEL_SOFTMAX, MODEL_MLP2, MODEL_SYNTH, MODEL_GIVEN = 0, 1, 2, 3, 4
FLAG_QUANT_OFF, FLAG_TRIGGER_OFF = 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "laq_oracle.cpp")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "liblaq_oracle.so")
_lib = None

_c_f32p = C.POINTER(C.c_float)
_c_f64p = C.POINTER(C.c_double)
_c_i32p = C.POINTER(C.c_int32)
_c_u32p = C.POINTER(C.c_uint32)
_c_i64p = C.POINTER(C.c_int64)


def build(force=False):
    """Compile the oracle if the shared object is missing or older than its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= os.path.getmtime(_SRC):
        return _SO
    tmp = _SO + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]
    try:  # explicit std::fma calls map to the hardware instruction where there is one (same result, faster)
        if " fma " in open("/proc/cpuinfo").read():
            cmd.append("-mfma")
    except OSError:
        pass
    cmd += ["-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _SO)
    return _SO


def _ptr(a, ty):
    return None if a is None else a.ctypes.data_as(ty)


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(build())
    L.laqo_quantize_f64.argtypes = [_c_f64p, _c_f64p, C.c_int64, C.c_int, _c_f64p, _c_i32p, _c_f64p,
                                    _c_f64p, _c_f64p, _c_f64p, _c_f64p]
    L.laqo_quantize_f32.argtypes = [_c_f32p, _c_f32p, C.c_int64, C.c_int, _c_f32p, _c_i32p, _c_f32p,
                                    _c_f32p, _c_f32p, _c_f64p, _c_f64p]
    L.laqo_decode_f64.argtypes = [C.c_double, _c_i32p, _c_f64p, C.c_int64, C.c_int, _c_f64p, _c_f64p]
    L.laqo_decode_f32.argtypes = [C.c_float, _c_i32p, _c_f32p, C.c_int64, C.c_int, _c_f32p, _c_f32p]
    L.laqo_code_words.argtypes = [C.c_int64, C.c_int]
    L.laqo_code_words.restype = C.c_int64
    L.laqo_pack_codes.argtypes = [_c_i32p, C.c_int64, C.c_int, _c_u32p]
    L.laqo_unpack_codes.argtypes = [_c_u32p, C.c_int64, C.c_int, _c_i32p]
    L.laqo_trigger.argtypes = [C.c_double, C.c_double, C.c_double, _c_f64p, _c_f32p, C.c_int,
                               C.c_float, C.c_int, C.c_int, C.c_int, C.c_int, _c_f64p]
    L.laqo_trigger.restype = C.c_int
    L.laqo_grad_logreg_bin.argtypes = [_c_f32p, _c_i32p, C.c_int64, C.c_int, _c_f64p, C.c_double,
                                       C.c_double, C.c_double, _c_f64p]
    L.laqo_grad_logreg_bin.restype = C.c_double
    L.laqo_grad_softmax.argtypes = [_c_f32p, _c_i32p, C.c_int64, C.c_int, C.c_int, _c_f64p,
                                    C.c_double, C.c_double, C.c_double, _c_f64p]
    L.laqo_grad_softmax.restype = C.c_double
    L.laqo_grad_mlp2.argtypes = [_c_f32p, _c_i32p, C.c_int64, C.c_int, C.c_int, C.c_int, _c_f64p,
                                 C.c_double, C.c_double, C.c_double, C.c_int, _c_f64p]
    L.laqo_grad_mlp2.restype = C.c_double
    L.laqo_synth_gradient.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_float,
                                      C.c_float, _c_f32p]
    L.laqo_round_bf16.argtypes = [C.c_float]
    L.laqo_round_bf16.restype = C.c_float
    L.laqo_new.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64, _c_i64p, C.c_int, C.c_int, C.c_int,
                           C.c_float, C.c_float, C.c_int, C.c_int, _c_f32p, C.c_int, C.c_int,
                           C.c_uint32, C.c_uint64, C.c_float, C.c_float, C.c_int, _c_f32p]
    L.laqo_new.restype = C.c_void_p
    L.laqo_free.argtypes = [C.c_void_p]
    L.laqo_set_batch.argtypes = [C.c_void_p, C.c_int]
    L.laqo_batch_offset.argtypes = [C.c_uint64, C.c_int, C.c_int64, C.c_int64]
    L.laqo_batch_offset.restype = C.c_int64
    L.laqo_set_shard.argtypes = [C.c_void_p, C.c_int, _c_f32p, _c_i32p, C.c_int64, C.c_int]
    L.laqo_set_shard.restype = C.c_int
    L.laqo_step.argtypes = [C.c_void_p]
    L.laqo_step_given.argtypes = [C.c_void_p, C.c_void_p]
    L.laqo_last_stats.argtypes = [C.c_void_p, _c_i32p, _c_f64p, _c_f64p, _c_f64p, _c_f64p, _c_f64p,
                                  _c_f64p, _c_f64p, _c_i32p]
    L.laqo_get_state.argtypes = [C.c_void_p, _c_f64p, _c_f64p, _c_f64p, _c_f64p, _c_i32p, _c_f64p,
                                 _c_i32p, _c_f64p, _c_i64p]
    L.laqo_set_state.argtypes = [C.c_void_p, _c_f64p, _c_f64p, _c_f64p, _c_f64p, _c_i32p, _c_f64p]
    L.laqo_loss.argtypes = [C.c_void_p]
    L.laqo_loss.restype = C.c_double
    _lib = L
    return L


# ------------------------------------------------------------------------------------------------
# stateless pieces
# ------------------------------------------------------------------------------------------------
def quantize(g, qp, b, dtype=np.float64):
    """Quantizer of Sec. 2.1 for one worker.  Returns a dict with R, q, dq, qnew, eps, n_dq, n_eps."""
    L = lib()
    dt = np.dtype(dtype)
    g = np.ascontiguousarray(g, dtype=dt)
    qp = np.ascontiguousarray(qp, dtype=dt)
    p = g.size
    R = np.zeros(1, dt)
    q = np.zeros(p, np.int32)
    dq, qnew, eps = np.zeros(p, dt), np.zeros(p, dt), np.zeros(p, dt)
    n_dq, n_eps = np.zeros(1), np.zeros(1)
    if dt == np.float64:
        L.laqo_quantize_f64(_ptr(g, _c_f64p), _ptr(qp, _c_f64p), p, b, _ptr(R, _c_f64p),
                            _ptr(q, _c_i32p), _ptr(dq, _c_f64p), _ptr(qnew, _c_f64p),
                            _ptr(eps, _c_f64p), _ptr(n_dq, _c_f64p), _ptr(n_eps, _c_f64p))
    else:
        L.laqo_quantize_f32(_ptr(g, _c_f32p), _ptr(qp, _c_f32p), p, b, _ptr(R, _c_f32p),
                            _ptr(q, _c_i32p), _ptr(dq, _c_f32p), _ptr(qnew, _c_f32p),
                            _ptr(eps, _c_f32p), _ptr(n_dq, _c_f64p), _ptr(n_eps, _c_f64p))
    return dict(R=R[0], q=q, dq=dq, qnew=qnew, eps=eps, n_dq=n_dq[0], n_eps=n_eps[0])


def decode(R, q, qp, b, dtype=np.float64):
    """Server-side recovery Q_new = Q_prev + (2 tau R q - R).  Returns (qnew, dq)."""
    L = lib()
    dt = np.dtype(dtype)
    q = np.ascontiguousarray(q, dtype=np.int32)
    qp = np.ascontiguousarray(qp, dtype=dt)
    qnew, dq = np.zeros(q.size, dt), np.zeros(q.size, dt)
    if dt == np.float64:
        L.laqo_decode_f64(float(R), _ptr(q, _c_i32p), _ptr(qp, _c_f64p), q.size, b,
                          _ptr(qnew, _c_f64p), _ptr(dq, _c_f64p))
    else:
        L.laqo_decode_f32(float(R), _ptr(q, _c_i32p), _ptr(qp, _c_f32p), q.size, b,
                          _ptr(qnew, _c_f32p), _ptr(dq, _c_f32p))
    return qnew, dq


def pack_codes(q, b):
    L = lib()
    q = np.ascontiguousarray(q, dtype=np.int32)
    words = np.zeros(L.laqo_code_words(q.size, b), np.uint32)
    L.laqo_pack_codes(_ptr(q, _c_i32p), q.size, b, _ptr(words, _c_u32p))
    return words


def unpack_codes(words, p, b):
    L = lib()
    words = np.ascontiguousarray(words, dtype=np.uint32)
    q = np.zeros(p, np.int32)
    L.laqo_unpack_codes(_ptr(words, _c_u32p), p, b, _ptr(q, _c_i32p))
    return q


def batch_offset(seed, m, k, n):
    """First sample of worker m's minibatch window at iteration k = 1, 2, .. (shard of n samples)."""
    return int(lib().laqo_batch_offset(int(seed), int(m), int(k), int(n)))


def trigger(n_dq, n_eps, n_epshat, dtheta2, xi, alpha, M, clock, tbar, clock_mode=0):
    """Eq. (7a)+(7b) for one worker; dtheta2[0] is the newest difference.  Returns (skip, rhs)."""
    L = lib()
    dtheta2 = np.ascontiguousarray(dtheta2, dtype=np.float64)
    xi = np.ascontiguousarray(xi, dtype=np.float32)
    rhs = np.zeros(1)
    s = L.laqo_trigger(n_dq, n_eps, n_epshat, _ptr(dtheta2, _c_f64p), _ptr(xi, _c_f32p), xi.size,
                       alpha, M, clock, tbar, clock_mode, _ptr(rhs, _c_f64p))
    return bool(s), rhs[0]


def _xy(X, y):
    X = np.ascontiguousarray(X, dtype=np.float32)
    y = np.ascontiguousarray(y, dtype=np.int32)
    return X, y


def grad_logreg_bin(X, y, theta, inv_N, share, lam):
    L = lib()
    X, y = _xy(X, y)
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    g = np.zeros(theta.size)
    loss = L.laqo_grad_logreg_bin(_ptr(X, _c_f32p), _ptr(y, _c_i32p), X.shape[0], X.shape[1],
                                  _ptr(theta, _c_f64p), inv_N, share, lam, _ptr(g, _c_f64p))
    return loss, g


def grad_softmax(X, y, theta, n_classes, inv_N, share, lam):
    L = lib()
    X, y = _xy(X, y)
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    g = np.zeros(theta.size)
    loss = L.laqo_grad_softmax(_ptr(X, _c_f32p), _ptr(y, _c_i32p), X.shape[0], X.shape[1], n_classes,
                               _ptr(theta, _c_f64p), inv_N, share, lam, _ptr(g, _c_f64p))
    return loss, g


def grad_mlp2(X, y, theta, n_hidden, n_classes, inv_N, share, lam, bf16_ops=0):
    L = lib()
    X, y = _xy(X, y)
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    g = np.zeros(theta.size)
    loss = L.laqo_grad_mlp2(_ptr(X, _c_f32p), _ptr(y, _c_i32p), X.shape[0], X.shape[1], n_hidden,
                            n_classes, _ptr(theta, _c_f64p), inv_N, share, lam, bf16_ops,
                            _ptr(g, _c_f64p))
    return loss, g


def synth_gradient(seed, m, M, p, k, sigma, eta0):
    L = lib()
    g = np.zeros(p, np.float32)
    L.laqo_synth_gradient(seed, m, M, p, k, sigma, eta0, _ptr(g, _c_f32p))
    return g


def lyapunov(losses, dtheta2s, xi, alpha, f_star):
    """Lyapunov function of Sec. 3, written out term by term:
        V(theta^k) = f(theta^k) - f(theta*) + sum_{d=1}^{D} sum_{j=d}^{D} (xi_j / alpha) ||theta^{k+1-d} - theta^{k-d}||^2.
    losses[k-1] = f(theta^k), dtheta2s[k-1] = ||theta^{k+1} - theta^k||^2 for k = 1..n; differences that lie before
    the first iteration do not exist and count as zero."""
    D, n = len(xi), len(losses)
    out = []
    for k in range(1, n + 1):
        v = float(losses[k - 1]) - float(f_star)
        for d in range(1, D + 1):
            it = k - d                      # ||theta^{k+1-d} - theta^{k-d}||^2 is the step of iteration k - d
            if it < 1:
                continue
            for j in range(d, D + 1):
                v += float(xi[j - 1]) / float(alpha) * float(dtheta2s[it - 1])
        out.append(v)
    return np.array(out)


def round_bf16(x):
    return lib().laqo_round_bf16(float(x))


# ------------------------------------------------------------------------------------------------
# the loop
# ------------------------------------------------------------------------------------------------
class OracleLaq:
    """Algorithm 2 with explicit state.  ``precision`` 64 = fp64 oracle, 32 = fp32 mirror."""

    def __init__(self, precision, model, M, p, N=None, n_features=0, n_classes=0, n_hidden=0,
                 alpha=0.02, lam=0.0, b=4, D=10, xi=None, tbar=100, clock_mode=0, flags=0, seed=0,
                 synth_sigma=0.1, synth_eta0=0.05, bf16_ops=0, theta0=None, batch=0):
        L = lib()
        self.L, self.precision, self.M, self.p, self.D, self.b = L, precision, M, int(p), D, b
        self.dtype = np.float64 if precision == 64 else np.float32
        N = np.ascontiguousarray(N if N is not None else np.zeros(M), dtype=np.int64)
        xi = np.ascontiguousarray(xi if xi is not None else np.full(D, 0.8 / max(D, 1)), np.float32)
        th0 = None if theta0 is None else np.ascontiguousarray(theta0, dtype=np.float32)
        self.h = L.laqo_new(precision, model, M, self.p, _ptr(N, _c_i64p), n_features, n_classes,
                            n_hidden, alpha, lam, b, D, _ptr(xi, _c_f32p), tbar, clock_mode, flags,
                            seed, synth_sigma, synth_eta0, bf16_ops, _ptr(th0, _c_f32p))
        if not self.h:
            raise ValueError("oracle rejected the configuration")

        if batch:
            L.laqo_set_batch(self.h, int(batch))

    def __del__(self):
        if getattr(self, "h", None):
            self.L.laqo_free(self.h)
            self.h = None

    def set_shard(self, m, X, y):
        X, y = _xy(X, y)
        rc = self.L.laqo_set_shard(self.h, m, _ptr(X, _c_f32p), _ptr(y, _c_i32p), X.shape[0], X.shape[1])
        if rc:
            raise ValueError("bad shard")

    def step(self):
        self.L.laqo_step(self.h)
        return self.last_stats()

    def step_given(self, g):
        g = np.ascontiguousarray(g, dtype=self.dtype)
        assert g.size == self.M * self.p
        self.L.laqo_step_given(self.h, g.ctypes.data_as(C.c_void_p))
        return self.last_stats()

    def last_stats(self):
        M = self.M
        skip, up = np.zeros(M, np.int32), np.zeros(1, np.int32)
        R, n_dq, n_eps, rhs, loss_m = (np.zeros(M) for _ in range(5))
        d2, loss = np.zeros(1), np.zeros(1)
        self.L.laqo_last_stats(self.h, _ptr(skip, _c_i32p), _ptr(R, _c_f64p), _ptr(n_dq, _c_f64p),
                               _ptr(n_eps, _c_f64p), _ptr(rhs, _c_f64p), _ptr(loss_m, _c_f64p),
                               _ptr(d2, _c_f64p), _ptr(loss, _c_f64p), _ptr(up, _c_i32p))
        return dict(skip=skip, R=R, n_dq=n_dq, n_eps=n_eps, rhs=rhs, loss_m=loss_m, dtheta2=d2[0],
                    loss=loss[0], uploads=int(up[0]))

    def state(self, big=True):
        M, p, D = self.M, self.p, self.D
        theta, agg = np.zeros(p), np.zeros(p)
        qp = np.zeros((M, p)) if big else None
        g = np.zeros((M, p)) if big else None
        codes = np.zeros((M, p), np.int32) if big else None
        n_epshat, clock, hist = np.zeros(M), np.zeros(M, np.int32), np.zeros(max(D, 1))
        cnt = np.zeros(3, np.int64)
        self.L.laqo_get_state(self.h, _ptr(theta, _c_f64p), _ptr(agg, _c_f64p), _ptr(qp, _c_f64p),
                              _ptr(g, _c_f64p), _ptr(codes, _c_i32p), _ptr(n_epshat, _c_f64p),
                              _ptr(clock, _c_i32p), _ptr(hist, _c_f64p), _ptr(cnt, _c_i64p))
        return dict(theta=theta, agg=agg, qp=qp, g=g, codes=codes, n_epshat=n_epshat, clock=clock,
                    hist=hist[:D], k=int(cnt[0]), uploads=int(cnt[1]), bits=int(cnt[2]))

    def set_state(self, theta=None, agg=None, qp=None, n_epshat=None, clock=None, hist=None):
        f64 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float64)
        theta, agg, qp, n_epshat, hist = map(f64, (theta, agg, qp, n_epshat, hist))
        clock = None if clock is None else np.ascontiguousarray(clock, dtype=np.int32)
        self.L.laqo_set_state(self.h, _ptr(theta, _c_f64p), _ptr(agg, _c_f64p), _ptr(qp, _c_f64p),
                              _ptr(n_epshat, _c_f64p), _ptr(clock, _c_i32p), _ptr(hist, _c_f64p))

    def loss(self):
        return self.L.laqo_loss(self.h)
