"""ctypes binding of libwersa.so: the same entry points as include/wersa.h, taking torch CUDA
tensors.  Argument marshalling only -- every step of the operator runs in the library's CUDA
kernels.  torch is used for device memory (the workspace) and streams.

The library must have been built (python -m paper_2507_08637_b200.build); importing this module
without it raises, there is no fallback."""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwersa.so")

WERSA_OK = 0
WERSA_F32, WERSA_BF16 = 0, 1
WERSA_FLAG_SIMT_ONLY = 1
WERSA_FLAG_FORWARD_ONLY = 2

STATUS_NAMES = ["WERSA_OK", "WERSA_ERR_INVALID_ARG", "WERSA_ERR_UNSUPPORTED", "WERSA_ERR_WORKSPACE",
                "WERSA_ERR_CUDA", "WERSA_ERR_TIMEOUT", "WERSA_ERR_STATE", "WERSA_ERR_TOO_LARGE"]


class wersa_config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("seq_len", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("levels", ctypes.c_int32), ("features", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("grad_dtype", ctypes.c_int32), ("eps", ctypes.c_float),
                ("bw_floor", ctypes.c_float), ("gate_per_head", ctypes.c_int32),
                ("device", ctypes.c_int32), ("flags", ctypes.c_int32)]


class WersaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name} ({_lib().wersa_status_string(status).decode()})")


_LIB = None


def _lib():
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2507_08637_b200.build` "
                          "(there is no non-CUDA fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, fp = ctypes.c_void_p, ctypes.c_void_p
    lib.wersa_workspace_bytes.restype = ctypes.c_size_t
    lib.wersa_workspace_bytes.argtypes = [ctypes.POINTER(wersa_config)]
    lib.wersa_create.restype = ctypes.c_int
    lib.wersa_create.argtypes = [ctypes.POINTER(wersa_config), vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.wersa_forward.restype = ctypes.c_int
    lib.wersa_forward.argtypes = [vp, vp, vp, vp, vp, fp, fp, fp, fp, vp, vp]
    lib.wersa_forward_host.restype = ctypes.c_int
    lib.wersa_forward_host.argtypes = [vp] + [vp] * 3 + [vp] * 3 + [vp] + [fp] * 4 + [vp, vp, vp]
    lib.wersa_backward.restype = ctypes.c_int
    lib.wersa_backward.argtypes = [vp] + [vp] * 4 + [fp] * 4 + [vp] * 4 + [fp] * 4 + [vp]
    lib.wersa_haar_filter.restype = ctypes.c_int
    lib.wersa_haar_filter.argtypes = [vp, vp, fp, vp, vp]
    lib.wersa_saved.restype = ctypes.c_int
    lib.wersa_saved.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
    lib.wersa_query_status.restype = ctypes.c_int
    lib.wersa_query_status.argtypes = [vp, vp]
    lib.wersa_destroy.restype = ctypes.c_int
    lib.wersa_destroy.argtypes = [vp]
    lib.wersa_status_string.restype = ctypes.c_char_p
    lib.wersa_status_string.argtypes = [ctypes.c_int]
    lib.wersa_launch_count.restype = ctypes.c_int32
    lib.wersa_launch_count.argtypes = [vp, ctypes.c_int]
    lib.wersa_gate_static.restype = ctypes.c_int
    lib.wersa_gate_static.argtypes = [ctypes.POINTER(wersa_config), vp, fp, fp, fp, fp, fp, vp]
    lib.wersa_shard_pool.restype = ctypes.c_int
    lib.wersa_shard_pool.argtypes = [vp, vp, vp, fp, vp]
    lib.wersa_shard_gate.restype = ctypes.c_int
    lib.wersa_shard_gate.argtypes = [vp, fp, ctypes.c_int64, fp, fp, fp, vp]
    lib.wersa_shard_keys.restype = ctypes.c_int
    lib.wersa_shard_keys.argtypes = [vp, vp, vp, vp]
    lib.wersa_shard_output.restype = ctypes.c_int
    lib.wersa_shard_output.argtypes = [vp, vp, fp, fp, fp, vp, vp]
    lib.wersa_shard_backward_queries.restype = ctypes.c_int
    lib.wersa_shard_backward_queries.argtypes = [vp, vp, fp, vp, vp]
    lib.wersa_shard_backward_keys.restype = ctypes.c_int
    lib.wersa_shard_backward_keys.argtypes = [vp, vp, vp, fp, fp, vp, vp, vp]
    lib.wersa_shard_backward_gate.restype = ctypes.c_int
    lib.wersa_shard_backward_gate.argtypes = [vp, fp, fp, ctypes.c_int64, fp, fp, fp, fp, fp, fp, fp, vp, vp]
    lib.wersa_selftest_wait_timeout.restype = ctypes.c_int
    lib.wersa_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint32, vp, vp]
    lib.wersa_uses_tensor_cores.restype = ctypes.c_int32
    lib.wersa_uses_tensor_cores.argtypes = [vp]
    lib.wersa_set_step_timing.restype = ctypes.c_int
    lib.wersa_set_step_timing.argtypes = [vp, ctypes.c_int]
    lib.wersa_step_times.restype = ctypes.c_int
    lib.wersa_step_times.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_float),
                                     ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_int)]
    _LIB = lib
    return lib


def _dtype_code(dt):
    if dt in ("f32", "fp32", torch.float32, WERSA_F32):
        return WERSA_F32
    if dt in ("bf16", torch.bfloat16, WERSA_BF16) and dt is not False:
        return WERSA_BF16
    raise ValueError(f"unsupported dtype {dt!r}")


def make_config(batch, heads, seq_len, head_dim, levels, features, dtype="bf16", grad_dtype="f32",
                eps=1e-6, bw_floor=1e-6, gate_per_head=1, device=0, flags=0):
    return wersa_config(batch, heads, seq_len, head_dim, levels, features, _dtype_code(dtype),
                        _dtype_code(grad_dtype), eps, bw_floor, int(gate_per_head), int(device), int(flags))


def wersa_workspace_bytes(cfg):
    return int(_lib().wersa_workspace_bytes(ctypes.byref(cfg)))


def wersa_status_string(status):
    return _lib().wersa_status_string(int(status)).decode()


def _ptr(t, dtype=None, name="tensor", optional=False):
    if t is None:
        if optional:
            return None
        raise ValueError(f"{name} is required")
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _host_ptr(t, dtype, name):
    if t is None or t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class WersaContext:
    """wersa_create / wersa_forward / wersa_backward / wersa_destroy around one workspace tensor."""

    def __init__(self, cfg):
        lib = _lib()
        self.cfg = cfg
        nbytes = int(lib.wersa_workspace_bytes(ctypes.byref(cfg)))
        if nbytes == 0:
            raise WersaError(2, "wersa_workspace_bytes (invalid or unsupported configuration)")
        self.device = torch.device("cuda", cfg.device)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        handle = ctypes.c_void_p()
        st = lib.wersa_create(ctypes.byref(cfg), ctypes.c_void_p(self.workspace.data_ptr()), nbytes,
                              ctypes.byref(handle))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_create")
        self._h = handle
        self.io_dtype = torch.bfloat16 if cfg.dtype == WERSA_BF16 else torch.float32
        self.grad_dtype = torch.bfloat16 if cfg.grad_dtype == WERSA_BF16 else torch.float32

    # -- entry points ---------------------------------------------------------------------
    def forward(self, Q, K, V, W, beta, gate_w, gate_b, omega, out=None, stream=None):
        if out is None:
            out = torch.empty_like(Q)
        dt = self.io_dtype
        st = _lib().wersa_forward(self._h, _ptr(Q, dt, "Q"), _ptr(K, dt, "K"), _ptr(V, dt, "V"),
                                  _ptr(W, dt, "W"), _ptr(beta, torch.float32, "beta"),
                                  _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                  _ptr(gate_b, torch.float32, "gate_b", optional=True),
                                  _ptr(omega, torch.float32, "omega"), _ptr(out, dt, "O"),
                                  _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_forward")
        return out

    def forward_host(self, hQ, hK, hV, dQ, dK, dV, W, beta, gate_w, gate_b, omega, dO, hO, stream=None):
        """wersa_forward_host: hQ, hK, hV, hO are contiguous HOST tensors (page-locked for asynchronous
        copies), dQ, dK, dV, dO device staging tensors of the same shape and dtype.  Everything is
        enqueued on `stream`; hO is valid once the stream has been synchronised."""
        dt = self.io_dtype
        st = _lib().wersa_forward_host(self._h, _host_ptr(hQ, dt, "hQ"), _host_ptr(hK, dt, "hK"),
                                       _host_ptr(hV, dt, "hV"), _ptr(dQ, dt, "dQ"), _ptr(dK, dt, "dK"),
                                       _ptr(dV, dt, "dV"), _ptr(W, dt, "W"), _ptr(beta, torch.float32, "beta"),
                                       _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                       _ptr(gate_b, torch.float32, "gate_b", optional=True),
                                       _ptr(omega, torch.float32, "omega"), _ptr(dO, dt, "dO"),
                                       _host_ptr(hO, dt, "hO"), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_forward_host")
        return hO

    def backward(self, Q, K, V, W, beta, gate_w, gate_b, omega, dO, stream=None):
        dt, gd = self.io_dtype, self.grad_dtype
        c = self.cfg
        dev = Q.device
        dQ = torch.empty(Q.shape, dtype=gd, device=dev)
        dK = torch.empty(Q.shape, dtype=gd, device=dev)
        dV = torch.empty(Q.shape, dtype=gd, device=dev)
        dbeta = torch.empty(1, dtype=torch.float32, device=dev)
        dgw = torch.empty((c.heads, c.head_dim, c.levels + 1), dtype=torch.float32, device=dev)
        dgb = torch.empty((c.heads, c.levels + 1), dtype=torch.float32, device=dev)
        dom = torch.empty(c.levels + 1, dtype=torch.float32, device=dev)
        st = _lib().wersa_backward(self._h, _ptr(Q, dt, "Q"), _ptr(K, dt, "K"), _ptr(V, dt, "V"),
                                   _ptr(W, dt, "W"), _ptr(beta, torch.float32, "beta"),
                                   _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                   _ptr(gate_b, torch.float32, "gate_b", optional=True),
                                   _ptr(omega, torch.float32, "omega"), _ptr(dO, dt, "dO"),
                                   _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dbeta), _ptr(dgw), _ptr(dgb),
                                   _ptr(dom), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_backward")
        return dict(dQ=dQ, dK=dK, dV=dV, dbeta=dbeta, dgate_w=dgw, dgate_b=dgb, domega=dom)

    def haar_filter(self, X, f, out=None, stream=None):
        if out is None:
            out = torch.empty_like(X)
        st = _lib().wersa_haar_filter(self._h, _ptr(X, self.io_dtype, "X"), _ptr(f, torch.float32, "f"),
                                      _ptr(out), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_haar_filter")
        return out

    # -- sequence-sharded forward: the four steps, the caller adds the sums of all shards in between --------
    def shard_pool(self, Q, W, stream=None):
        qsum = torch.empty((self.cfg.batch, self.cfg.heads, 64), dtype=torch.float32, device=self.device)
        st = _lib().wersa_shard_pool(self._h, _ptr(Q, self.io_dtype, "Q"), _ptr(W, self.io_dtype, "W"), _ptr(qsum),
                                     _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_pool")
        return qsum

    def shard_gate(self, qsum_total, n_total, gate_w, gate_b, omega, stream=None):
        st = _lib().wersa_shard_gate(self._h, _ptr(qsum_total, torch.float32, "qsum_total"), int(n_total),
                                     _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                     _ptr(gate_b, torch.float32, "gate_b", optional=True),
                                     _ptr(omega, torch.float32, "omega"), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_gate")

    def shard_keys(self, K, V, stream=None):
        """Returns views of this shard's S' (batch, heads, features, 64) and z' in the workspace."""
        st = _lib().wersa_shard_keys(self._h, _ptr(K, self.io_dtype, "K"), _ptr(V, self.io_dtype, "V"),
                                     _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_keys")
        return self._saved_view(2), self._saved_view(3)

    def shard_output(self, Q, S_total, z_total, beta, out=None, stream=None):
        if out is None:
            out = torch.empty_like(Q)
        st = _lib().wersa_shard_output(self._h, _ptr(Q, self.io_dtype, "Q"), _ptr(S_total, torch.float32, "S_total"),
                                       _ptr(z_total, torch.float32, "z_total"), _ptr(beta, torch.float32, "beta"),
                                       _ptr(out, self.io_dtype, "O"), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_output")
        return out

    def shard_backward_queries(self, Q, beta, dO, stream=None):
        """Returns views of this shard's dS' and dz' in the workspace."""
        st = _lib().wersa_shard_backward_queries(self._h, _ptr(Q, self.io_dtype, "Q"), _ptr(beta, torch.float32, "beta"),
                                                 _ptr(dO, self.io_dtype, "dO"), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_backward_queries")
        return self._saved_view(4), self._saved_view(5)

    def shard_backward_keys(self, K, V, dS_total, dz_total, stream=None):
        """Returns dK, dV of this shard and views of its band inner products and its sum of dD'."""
        dK = torch.empty(K.shape, dtype=self.grad_dtype, device=self.device)
        dV = torch.empty(K.shape, dtype=self.grad_dtype, device=self.device)
        st = _lib().wersa_shard_backward_keys(self._h, _ptr(K, self.io_dtype, "K"), _ptr(V, self.io_dtype, "V"),
                                              _ptr(dS_total, torch.float32, "dS_total"),
                                              _ptr(dz_total, torch.float32, "dz_total"), _ptr(dK), _ptr(dV),
                                              _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_backward_keys")
        return dK, dV, self._saved_view(6), self._saved_view(7)

    def shard_backward_gate(self, Q, df_total, sumdD_total, n_total, beta, gate_w, omega, stream=None):
        """Returns dict(dQ, dbeta, dgate_w, dgate_b, domega) for this shard (the parameter gradients are the
        same on every rank)."""
        c, dev = self.cfg, self.device
        dQ = torch.empty(Q.shape, dtype=self.grad_dtype, device=dev)
        dbeta = torch.empty(1, dtype=torch.float32, device=dev)
        dgw = torch.empty((c.heads, c.head_dim, c.levels + 1), dtype=torch.float32, device=dev)
        dgb = torch.empty((c.heads, c.levels + 1), dtype=torch.float32, device=dev)
        dom = torch.empty(c.levels + 1, dtype=torch.float32, device=dev)
        st = _lib().wersa_shard_backward_gate(self._h, _ptr(df_total, torch.float32, "df_total"),
                                              _ptr(sumdD_total, torch.float32, "sumdD_total"), int(n_total),
                                              _ptr(beta, torch.float32, "beta"),
                                              _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                              _ptr(omega, torch.float32, "omega"), _ptr(dbeta), _ptr(dgw), _ptr(dgb),
                                              _ptr(dom), _ptr(dQ), _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_shard_backward_gate")
        return dict(dQ=dQ, dbeta=dbeta, dgate_w=dgw, dgate_b=dgb, domega=dom)

    def _saved_view(self, idx):
        ptr, count = ctypes.c_void_p(), ctypes.c_size_t()
        st = _lib().wersa_saved(self._h, idx, ctypes.byref(ptr), ctypes.byref(count))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_saved")
        off = ptr.value - self.workspace.data_ptr()
        c = self.cfg
        shape = {2: (c.batch, c.heads, c.features, 64), 3: (c.batch, c.heads, c.features),
                 4: (c.batch, c.heads, c.features, 64), 5: (c.batch, c.heads, c.features),
                 6: (c.batch, c.heads, 16), 7: (1,)}[idx]
        return self.workspace[off:off + 4 * count.value].view(torch.float32).view(shape)

    def saved(self, which):
        """Copy of a tensor the last forward left in the workspace: 'f', 'qbar', 'S', 'z'."""
        idx = {"f": 0, "qbar": 1, "S": 2, "z": 3}[which]
        ptr, count = ctypes.c_void_p(), ctypes.c_size_t()
        st = _lib().wersa_saved(self._h, idx, ctypes.byref(ptr), ctypes.byref(count))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_saved")
        off = ptr.value - self.workspace.data_ptr()
        flat = self.workspace[off:off + 4 * count.value].view(torch.float32).clone()
        c = self.cfg
        slabs = (c.batch, c.heads)
        shape = {0: slabs + (c.levels + 1,), 1: slabs + (64,), 2: slabs + (c.features, 64),
                 3: slabs + (c.features,)}[idx]
        out = flat.view(shape)
        return out[..., :c.head_dim].contiguous() if idx in (1, 2) else out   # drop the padding columns

    def query_status(self, stream=None):
        return int(_lib().wersa_query_status(self._h, _stream_ptr(stream)))

    def selftest_wait_timeout(self, limit_us=1000, stream=None):
        """wersa_selftest_wait_timeout: returns the three ints the kernel observed (abort flag, and whether
        the two roles' waits succeeded) as a CUDA int32 tensor; read it after synchronising."""
        observed = torch.full((3,), -1, dtype=torch.int32, device=self.device)
        st = _lib().wersa_selftest_wait_timeout(self._h, int(limit_us), _ptr(observed, torch.int32, "observed"),
                                                _stream_ptr(stream))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_selftest_wait_timeout")
        return observed

    def set_step_timing(self, enable):
        st = _lib().wersa_set_step_timing(self._h, int(bool(enable)))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_set_step_timing")

    def step_times(self, which=0):
        """[(step name, milliseconds)] of the last forward (0) or backward (1); waits for it."""
        cap = 32
        ms = (ctypes.c_float * cap)()
        names = (ctypes.c_char_p * cap)()
        count = ctypes.c_int()
        st = _lib().wersa_step_times(self._h, which, cap, ms, names, ctypes.byref(count))
        if st != WERSA_OK:
            raise WersaError(st, "wersa_step_times")
        return [(names[i].decode(), float(ms[i])) for i in range(min(count.value, cap))]

    def uses_tensor_cores(self):
        return bool(_lib().wersa_uses_tensor_cores(self._h))

    def launch_count(self, which=0):
        return int(_lib().wersa_launch_count(self._h, which))

    def destroy(self):
        if getattr(self, "_h", None) is not None:
            _lib().wersa_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def wersa_create(batch, heads, seq_len, head_dim, levels, features, **kw):
    return WersaContext(make_config(batch, heads, seq_len, head_dim, levels, features, **kw))


def wersa_forward(ctx, Q, K, V, W, beta, gate_w, gate_b, omega, out=None, stream=None):
    return ctx.forward(Q, K, V, W, beta, gate_w, gate_b, omega, out=out, stream=stream)


def wersa_forward_host(ctx, hQ, hK, hV, dQ, dK, dV, W, beta, gate_w, gate_b, omega, dO, hO, stream=None):
    return ctx.forward_host(hQ, hK, hV, dQ, dK, dV, W, beta, gate_w, gate_b, omega, dO, hO, stream=stream)


def wersa_backward(ctx, Q, K, V, W, beta, gate_w, gate_b, omega, dO, stream=None):
    return ctx.backward(Q, K, V, W, beta, gate_w, gate_b, omega, dO, stream=stream)


def wersa_destroy(ctx):
    ctx.destroy()


def wersa_gate_static(cfg, Q, gate_w, gate_b, omega, qbar, f, stream=None):
    """Mean-pooled query and gate without a context or workspace, for callers that cannot
    allocate device memory when they need the gate (a frozen or foreign allocator, memory fully
    committed): the library's own fixed 1 MiB device array holds the intermediate sums.  The
    caller passes the outputs qbar (batch*heads, head_dim) and f (batch*heads, levels+1), float32
    CUDA tensors; nothing is allocated here or in the library.  Raises WersaError with status
    WERSA_ERR_TOO_LARGE when the problem does not fit the fixed array.  Calls that may overlap on
    the GPU must be serialised by the caller; make the first call on a device outside stream
    capture."""
    io = torch.bfloat16 if cfg.dtype == WERSA_BF16 else torch.float32
    st = _lib().wersa_gate_static(ctypes.byref(cfg), _ptr(Q, io, "Q"),
                                  _ptr(gate_w, torch.float32, "gate_w", optional=True),
                                  _ptr(gate_b, torch.float32, "gate_b", optional=True),
                                  _ptr(omega, torch.float32, "omega"), _ptr(qbar, torch.float32, "qbar"),
                                  _ptr(f, torch.float32, "f"), _stream_ptr(stream))
    if st != WERSA_OK:
        raise WersaError(st, "wersa_gate_static")
