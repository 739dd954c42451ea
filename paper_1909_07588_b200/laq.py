"""Thin ctypes binding of the C ABI in ``include/laq.h`` (argument marshalling only).

PyTorch supplies device memory and the stream; every step of the LAQ iteration runs inside
``csrc/liblaq_b200.so``.  If that library is missing this module raises -- there is no fallback.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "liblaq_b200.so")

LAQ_OK, LAQ_EINVAL, LAQ_EWORKSPACE, LAQ_ECUDA, LAQ_ENONFINITE, LAQ_ESTATE, LAQ_ETIMEOUT = range(7)
STATUS_NAMES = ["LAQ_OK", "LAQ_EINVAL", "LAQ_EWORKSPACE", "LAQ_ECUDA", "LAQ_ENONFINITE", "LAQ_ESTATE", "LAQ_ETIMEOUT"]
MODEL_LOGREG_BIN, MODEL_SOFTMAX, MODEL_MLP2, MODEL_SYNTH, MODEL_EXTERNAL = range(5)
FLAG_QUANT_OFF = 1
FLAG_TRIGGER_OFF = 2
FLAG_STORE_G = 4
FLAG_SPARSE_X = 8

EXPORTS = ["laq_workspace_bytes", "laq_init", "laq_load_shards", "laq_set_gradients", "laq_step", "laq_step_local", "laq_local_uploads", "laq_apply_uploads", "laq_sync",
           "laq_get_state", "laq_get_worker", "laq_set_state", "laq_kernel_launches", "laq_tune", "laq_query", "laq_set_profiling", "laq_kernel_times", "laq_quantize_worker_static", "laq_last_error", "laq_destroy"]


class LaqError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status, message))
        self.status = status


class laq_config(C.Structure):
    _fields_ = [("model", C.c_int32), ("M", C.c_int32), ("p", C.c_int64), ("N", C.POINTER(C.c_int64)),
                ("n_features", C.c_int32), ("n_classes", C.c_int32), ("n_hidden", C.c_int32),
                ("alpha", C.c_float), ("lam", C.c_float), ("b", C.c_int32), ("D", C.c_int32),
                ("xi", C.POINTER(C.c_float)), ("tbar", C.c_int32), ("clock_mode", C.c_int32),
                ("flags", C.c_uint32), ("seed", C.c_uint64), ("synth_sigma", C.c_float),
                ("synth_eta0", C.c_float), ("trace_capacity", C.c_int32), ("batch", C.c_int32),
                ("world", C.c_int32), ("rank", C.c_int32)]


class laq_trace(C.Structure):
    _fields_ = [("skip", C.c_void_p), ("R", C.c_void_p), ("n_dq", C.c_void_p), ("n_eps", C.c_void_p),
                ("rhs", C.c_void_p), ("dtheta2", C.c_void_p), ("loss", C.c_void_p), ("uploads", C.c_void_p)]


class laq_state(C.Structure):
    _fields_ = [("theta", C.c_void_p), ("agg", C.c_void_p), ("qprev", C.c_void_p), ("n_eps_hat", C.c_void_p),
                ("clock", C.c_void_p), ("ring", C.c_void_p), ("counters", C.c_void_p), ("g", C.c_void_p),
                ("codes", C.c_void_p), ("R", C.c_void_p), ("n_dq", C.c_void_p), ("n_eps", C.c_void_p),
                ("skip", C.c_void_p)]


_lib = None


def load_library():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("CUDA library %s is missing: run `python -m paper_1909_07588_b200.build` "
                          "(there is no CPU fallback)" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    L.laq_workspace_bytes.argtypes = [C.POINTER(laq_config)]
    L.laq_workspace_bytes.restype = C.c_size_t
    L.laq_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(laq_config), C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    L.laq_load_shards.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32]
    L.laq_set_gradients.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
    L.laq_step.argtypes = [C.c_void_p, C.c_int32, C.POINTER(laq_trace)]
    L.laq_step_local.argtypes = [C.c_void_p]
    L.laq_local_uploads.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_void_p, C.c_void_p]
    L.laq_apply_uploads.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.laq_sync.argtypes = [C.c_void_p]
    L.laq_get_state.argtypes = [C.c_void_p, C.POINTER(laq_state)]
    L.laq_set_state.argtypes = [C.c_void_p, C.POINTER(laq_state)]
    L.laq_get_worker.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.laq_kernel_launches.argtypes = [C.c_void_p]
    L.laq_kernel_launches.restype = C.c_int64
    L.laq_tune.argtypes = [C.c_void_p, C.c_char_p, C.c_int32]
    L.laq_query.argtypes = [C.c_void_p, C.c_char_p, C.POINTER(C.c_int64)]
    L.laq_set_profiling.argtypes = [C.c_void_p, C.c_int32]
    L.laq_kernel_times.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    L.laq_quantize_worker_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_char_p, C.c_size_t]
    L.laq_last_error.argtypes = [C.c_void_p]
    L.laq_last_error.restype = C.c_char_p
    L.laq_destroy.argtypes = [C.c_void_p]
    L.laq_destroy.restype = None
    _lib = L
    return L


def make_config(model, M, p, N=None, n_features=0, n_classes=0, n_hidden=0, alpha=0.02, lam=0.0, b=4, D=10,
                xi=None, tbar=100, clock_mode=0, flags=0, seed=0, synth_sigma=0.1, synth_eta0=0.05,
                trace_capacity=0, batch=0, world=0, rank=0):
    """Returns (laq_config, keepalive) -- keepalive holds the numpy arrays the struct points to."""
    N_arr = np.ascontiguousarray(N if N is not None else np.zeros(max(M, 1)), dtype=np.int64)
    xi_arr = np.ascontiguousarray(xi if xi is not None else np.full(max(D, 1), 0.8 / max(D, 1)), dtype=np.float32)
    cfg = laq_config(model, M, p, N_arr.ctypes.data_as(C.POINTER(C.c_int64)), n_features, n_classes, n_hidden,
                     alpha, lam, b, D, xi_arr.ctypes.data_as(C.POINTER(C.c_float)), tbar, clock_mode, flags,
                     seed, synth_sigma, synth_eta0, trace_capacity, batch, world, rank)
    return cfg, (N_arr, xi_arr)


def workspace_bytes(cfg):
    return int(load_library().laq_workspace_bytes(C.byref(cfg)))


def _np_ptr(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


class Laq:
    """One LAQ context on the current CUDA device.  Mirrors laq_init / laq_load_shards / laq_step /
    laq_get_state / laq_destroy; the device workspace is a torch uint8 tensor owned by this object."""

    def __init__(self, stream=None, device=None, **config):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_1909_07588_b200.Laq needs a CUDA device (there is no CPU fallback)")
        self._L = load_library()
        self._torch = torch
        self.device = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
        self.theta0 = config.pop("theta0", None)
        self.cfg, self._keep = make_config(**config)
        # per-worker arrays of a context have one row per LOCAL worker (all M unless the workers are spread over
        # several contexts with world > 1); M_total keeps the global count
        self.M_total, self.world, self.rank = self.cfg.M, max(self.cfg.world, 1), self.cfg.rank
        self.M = (self.M_total - self.rank + self.world - 1) // self.world
        self.p, self.D, self.b = int(self.cfg.p), self.cfg.D, self.cfg.b
        self.model = self.cfg.model
        self.trace_capacity = self.cfg.trace_capacity
        nbytes = workspace_bytes(self.cfg)
        if nbytes == 0:
            # let laq_init produce the message
            nbytes = 256
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            th0 = None if self.theta0 is None else np.ascontiguousarray(self.theta0, dtype=np.float32)
            h = C.c_void_p()
            st = self._L.laq_init(C.byref(h), C.byref(self.cfg), C.c_void_p(self.workspace.data_ptr()), nbytes,
                                  _np_ptr(th0), C.c_void_p(self.stream.cuda_stream))
        self._h = h
        if st != LAQ_OK:
            msg = self._L.laq_last_error(h).decode() if h else "laq_init failed"
            self._L.laq_destroy(h)
            self._h = None
            raise LaqError(st, msg)

    # -- helpers ---------------------------------------------------------------------------------
    def _check(self, st):
        if st != LAQ_OK:
            raise LaqError(st, self._L.laq_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self._L.laq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI -----------------------------------------------------------------------------------
    def load_shards(self, m, X, y):
        """X: [N_m, F] fp32, y: [N_m] int32; numpy arrays (host) or torch CUDA tensors (device)."""
        torch = self._torch
        if isinstance(X, torch.Tensor):
            assert X.is_cuda and y.is_cuda and X.dtype == torch.float32 and y.dtype == torch.int32
            X, y = X.contiguous(), y.contiguous()
            st = self._L.laq_load_shards(self._h, m, C.c_void_p(X.data_ptr()), C.c_void_p(y.data_ptr()), X.shape[0], 1)
        else:
            X = np.ascontiguousarray(X, dtype=np.float32)
            y = np.ascontiguousarray(y, dtype=np.int32)
            st = self._L.laq_load_shards(self._h, m, _np_ptr(X), _np_ptr(y), X.shape[0], 0)
        self._check(st)

    def set_gradients(self, g):
        torch = self._torch
        if isinstance(g, torch.Tensor):
            assert g.is_cuda and g.dtype == torch.float32 and g.numel() == self.M * self.p
            g = g.contiguous()
            st = self._L.laq_set_gradients(self._h, C.c_void_p(g.data_ptr()), 1)
        else:
            g = np.ascontiguousarray(g, dtype=np.float32)
            assert g.size == self.M * self.p
            st = self._L.laq_set_gradients(self._h, _np_ptr(g), 0)
        self._check(st)

    def step(self, n_iters=1, trace=False):
        """Runs n_iters iterations.  With trace=True returns a dict of per-iteration host arrays."""
        if not trace:
            self._check(self._L.laq_step(self._h, n_iters, None))
            return None
        n, M = n_iters, self.M
        out = dict(skip=np.zeros((n, M), np.uint8), R=np.zeros((n, M), np.float32), n_dq=np.zeros((n, M)),
                   n_eps=np.zeros((n, M)), rhs=np.zeros((n, M)), dtheta2=np.zeros(n), loss=np.zeros(n),
                   uploads=np.zeros(n, np.int32))
        tr = laq_trace(*[_np_ptr(out[k]) for k in ("skip", "R", "n_dq", "n_eps", "rhs", "dtheta2", "loss", "uploads")])
        self._check(self._L.laq_step(self._h, n_iters, C.byref(tr)))
        return out

    def sync(self):
        self._check(self._L.laq_sync(self._h))

    # -- one iteration in two halves (workers spread over several contexts) ------------------------
    def step_local(self):
        """Steps 1-4 for this context's workers (enqueue only)."""
        self._check(self._L.laq_step_local(self._h))

    def local_uploads(self):
        """(global worker indices, radii) of the local uploaders of the iteration in flight (synchronises)."""
        n = C.c_int32(0)
        m, R = np.zeros(max(self.M, 1), np.int32), np.zeros(max(self.M, 1), np.float32)
        self._check(self._L.laq_local_uploads(self._h, C.byref(n), _np_ptr(m), _np_ptr(R)))
        return m[:n.value].copy(), R[:n.value].copy()

    def apply_uploads(self, m, R):
        """Step 5 with all uploads of the iteration: global worker indices (ascending) and radii."""
        m = np.ascontiguousarray(m, dtype=np.int32)
        R = np.ascontiguousarray(R, dtype=np.float32)
        assert m.size == R.size
        self._check(self._L.laq_apply_uploads(self._h, int(m.size), _np_ptr(m), _np_ptr(R)))

    def code_row(self, local_worker):
        """The code stream of a LOCAL worker's message as a view (int32 words) into the workspace."""
        off, row = self.query("codes_offset_bytes"), self.query("code_row_bytes")
        a = off + local_worker * row
        return self.workspace[a:a + row].view(self._torch.int32)

    def mailbox_row(self, global_worker):
        """Where the code stream of a REMOTE worker's message must be put before apply_uploads (view, int32 words)."""
        off, row = self.query("mailbox_offset_bytes"), self.query("code_row_bytes")
        assert off >= 0, "this context holds all workers: it has no mailbox"
        a = off + global_worker * row
        return self.workspace[a:a + row].view(self._torch.int32)

    def get_state(self, big=True, g=False, codes=False, agg=True, buffers=None):
        """Copies state to host arrays (synchronises).  big / g / codes / agg select the large fields;
        ``buffers`` may supply the destination arrays by field name (e.g. views of pinned host memory, which the
        copies then land in at PCIe speed); the others are allocated here."""
        M, p, D = self.M, self.p, self.D
        W = (p * self.b + 31) // 32
        out = dict(theta=np.zeros(p, np.float32) if not (buffers and "theta" in buffers) else buffers["theta"],
                   agg=(np.zeros(p, np.float32) if not (buffers and "agg" in buffers) else buffers["agg"]) if agg else None,
                   qprev=np.zeros((M, p), np.float32) if big else None,
                   n_eps_hat=np.zeros(M), clock=np.zeros(M, np.int32), ring=np.zeros(D), counters=np.zeros(3, np.int64),
                   g=np.zeros((M, p), np.float32) if g else None,
                   codes=np.zeros((M, W), np.uint32) if codes else None,
                   R=np.zeros(M, np.float32), n_dq=np.zeros(M), n_eps=np.zeros(M), skip=np.zeros(M, np.uint8))
        assert out["theta"].dtype == np.float32 and out["theta"].size == p and out["theta"].flags["C_CONTIGUOUS"]
        st = laq_state(*[_np_ptr(out[k]) for k in ("theta", "agg", "qprev", "n_eps_hat", "clock", "ring", "counters",
                                                   "g", "codes", "R", "n_dq", "n_eps", "skip")])
        self._check(self._L.laq_get_state(self._h, C.byref(st)))
        out["k"], out["uploads"], out["bits"] = (int(v) for v in out["counters"])
        return out

    def get_worker(self, m, qprev=True, g=False, codes=True):
        """One worker's rows: dict with qprev [p], g [p], codes [W] (the message's code stream) and R."""
        p, W = self.p, (self.p * self.b + 31) // 32
        out = dict(qprev=np.zeros(p, np.float32) if qprev else None, g=np.zeros(p, np.float32) if g else None,
                   codes=np.zeros(W, np.uint32) if codes else None, R=np.zeros(1, np.float32))
        self._check(self._L.laq_get_worker(self._h, m, _np_ptr(out["qprev"]), _np_ptr(out["g"]),
                                           _np_ptr(out["codes"]), _np_ptr(out["R"])))
        out["R"] = out["R"][0]
        return out

    def set_state(self, theta=None, agg=None, qprev=None, n_eps_hat=None, clock=None, ring=None, counters=None):
        conv = lambda a, dt: None if a is None else np.ascontiguousarray(a, dtype=dt)
        arrs = dict(theta=conv(theta, np.float32), agg=conv(agg, np.float32), qprev=conv(qprev, np.float32),
                    n_eps_hat=conv(n_eps_hat, np.float64), clock=conv(clock, np.int32), ring=conv(ring, np.float64),
                    counters=conv(counters, np.int64))
        st = laq_state(*([_np_ptr(arrs[k]) for k in ("theta", "agg", "qprev", "n_eps_hat", "clock", "ring", "counters")]
                         + [None] * 6))
        self._check(self._L.laq_set_state(self._h, C.byref(st)))

    def kernel_launches(self):
        return int(self._L.laq_kernel_launches(self._h))

    def set_profiling(self, enabled):
        self._check(self._L.laq_set_profiling(self._h, 1 if enabled else 0))

    def kernel_times(self):
        """(ms[4], launches[4]) per stage since the last call: gradient, radius, quantize+trigger, aggregate."""
        ms, n = np.zeros(4), np.zeros(4, np.int64)
        self._check(self._L.laq_kernel_times(self._h, _np_ptr(ms), _np_ptr(n)))
        return ms, n

    def tune(self, key, value):
        self._check(self._L.laq_tune(self._h, key.encode(), int(value)))

    def query(self, key):
        v = C.c_int64(0)
        st = self._L.laq_query(self._h, key.encode(), C.byref(v))
        if st != LAQ_OK:
            raise LaqError(st, "unknown query key %r" % key)
        return int(v.value)


def from_workload(w, trace_capacity=0, stream=None, **overrides):
    """Build a context from a ``workloads.Workload`` and make its shards resident."""
    kw = dict(model=w.model, M=w.M, p=w.p, N=w.N, n_features=w.n_features, n_classes=w.n_classes,
              n_hidden=w.n_hidden, alpha=w.alpha, lam=w.lam, b=w.b, D=w.D, xi=w.xi, tbar=w.tbar, seed=w.seed,
              synth_sigma=w.synth_sigma, synth_eta0=w.synth_eta0, trace_capacity=trace_capacity, theta0=w.theta0)
    kw.update(overrides)
    ctx = Laq(stream=stream, **kw)
    world, rank = max(kw.get("world", 0), 1), kw.get("rank", 0)
    for l, m in enumerate(range(rank, len(w.X), world)):      # shards of the local workers, by local index
        ctx.load_shards(l, w.X[m], w.y[m])
    return ctx


def quantize_worker_static(g, qprev, b, codes, R, norms, stream=None):
    """laq_quantize_worker_static: one worker's quantizer for hosts that must not allocate device memory.

    Every argument is a torch CUDA tensor that the caller already owns: g, qprev [p] float32 (inputs),
    codes [ceil(p*b/32)] int32 or uint32 storage, R [1] float32, norms [2] float64 (outputs).  The kernels'
    scratch is a fixed array inside the library, shared by all calls on the GPU, so calls must not overlap.
    """
    import torch
    L = load_library()
    assert g.is_cuda and qprev.is_cuda and codes.is_cuda and R.is_cuda and norms.is_cuda
    assert g.dtype == torch.float32 and qprev.dtype == torch.float32 and R.dtype == torch.float32
    assert norms.dtype == torch.float64 and norms.numel() >= 2 and codes.element_size() == 4
    p = g.numel()
    assert qprev.numel() == p and codes.numel() >= (p * b + 31) // 32
    err = C.create_string_buffer(256)
    with torch.cuda.device(g.device):        # the library uses the scratch of the calling thread's current device
        st = stream if stream is not None else torch.cuda.current_stream(g.device)
        rc = L.laq_quantize_worker_static(C.c_void_p(g.data_ptr()), C.c_void_p(qprev.data_ptr()), p, b,
                                          C.c_void_p(codes.data_ptr()), C.c_void_p(R.data_ptr()),
                                          C.c_void_p(norms.data_ptr()), C.c_void_p(st.cuda_stream), err, 256)
    if rc != LAQ_OK:
        raise LaqError(rc, err.value.decode())
