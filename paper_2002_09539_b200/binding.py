"""ctypes binding of libolsgd: argument marshalling only.

Every step of the method runs in the library's CUDA kernels.  There is no CPU
fallback: if the shared library is missing or cannot be loaded, importing a
symbol from it raises.
"""
import ctypes as C
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB = None

KERNEL_CLASSES = ("index", "gather", "forward", "backward", "update", "anchor", "loss", "other",
                  "wgrad_update")
_KINDS = {"linreg": 0, "softmax": 1, "mlp": 2, "flat": 3}
MAX_DIMS = 8


class OlsgdError(RuntimeError):
    def __init__(self, status, text):
        super().__init__("olsgd status %d: %s" % (status, text))
        self.status = status


class _ModelSpec(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_dims", C.c_int32), ("dims", C.c_int32 * MAX_DIMS),
                ("gemm_bf16", C.c_int32), ("reserved", C.c_int32), ("flat_P", C.c_int64)]


class _HParams(C.Structure):
    _fields_ = [("m", C.c_int32), ("tau", C.c_int32), ("batch", C.c_int32), ("mode", C.c_int32),
                ("gamma", C.c_float), ("alpha", C.c_float), ("beta", C.c_float), ("mu", C.c_float),
                ("seed", C.c_uint64), ("worker_offset", C.c_int32), ("m_total", C.c_int32),
                ("sampling", C.c_int32), ("reserved2", C.c_int32)]


class _Data(C.Structure):
    _fields_ = [("X", C.c_void_p), ("y", C.c_void_p), ("n_per_worker", C.c_int64)]


def lib_path():
    return os.path.join(_PKG, "libolsgd.so")


def load_library():
    """Load libolsgd.so (built by `python -m paper_2002_09539_b200.build`)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError("libolsgd.so is not built; run python -m paper_2002_09539_b200.build")
    lib = C.CDLL(path)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    sig = {
        "olsgd_param_count": (i32, [C.POINTER(_ModelSpec), C.POINTER(i64)]),
        "olsgd_workspace_bytes": (i32, [C.POINTER(_ModelSpec), C.POINTER(_HParams),
                                        C.POINTER(C.c_size_t)]),
        "olsgd_init": (i32, [C.POINTER(vp), C.POINTER(_ModelSpec), C.POINTER(_HParams),
                             C.POINTER(_Data), vp, vp, C.c_size_t, vp, vp]),
        "olsgd_local_step": (i32, [vp, vp]),
        "olsgd_local_step_with_grads": (i32, [vp, vp]),
        "olsgd_local_step_host": (i32, [vp, vp, vp, vp]),
        "olsgd_local_step_host_bf16": (i32, [vp, vp, vp, vp]),
        "olsgd_join": (i32, [vp]),
        "olsgd_selftest_wait_timeout": (i32, [vp, i32]),
        "olsgd_clear_status": (i32, [vp]),
        "olsgd_selftest_per_device_table": (i32, []),
        "olsgd_epoch_rule_half_bits": (i32, [i64]),
        "olsgd_period_sync": (i32, [vp]),
        "olsgd_set_anchor_fusion": (i32, [vp, i32]),
        "olsgd_anchor_fusion": (i32, [vp]),
        "olsgd_summed_floats": (i64, [vp]),
        "olsgd_period_sync_begin": (i32, [vp, vp]),
        "olsgd_period_sync_finish": (i32, [vp, vp]),
        "olsgd_row_floats": (i64, [vp]),
        "olsgd_run": (i32, [vp, i64, vp]),
        "olsgd_get_params": (i32, [vp, i32, vp, C.c_size_t]),
        "olsgd_get_indices": (i32, [vp, i64, vp]),
        "olsgd_set_params": (i32, [vp, i32, vp, C.c_size_t]),
        "olsgd_set_iteration": (i32, [vp, i64]),
        "olsgd_consensus_distance": (i32, [vp, C.POINTER(C.c_double)]),
        "olsgd_class_pairs": (i32, [u64, i32, vp, vp]),
        "olsgd_class_pairs_noalloc": (i32, [u64, i32, vp, vp]),
        "olsgd_iteration": (i64, [vp]),
        "olsgd_launch_count": (i64, [vp]),
        "olsgd_graph_replays": (i64, [vp]),
        "olsgd_graph_block": (i64, [vp]),
        "olsgd_set_launch_overlap": (i32, [i32]),
        "olsgd_set_gemm_pairs": (i32, [i32]),
        "olsgd_tensor_core_launches": (i64, []),
        "olsgd_profile_enable": (i32, [vp, i32]),
        "olsgd_profile_read": (i32, [vp, C.POINTER(i64), C.POINTER(C.c_double), i32]),
        "olsgd_profile_read_layers": (i32, [vp, C.POINTER(i64), C.POINTER(C.c_double), i32]),
        "olsgd_last_error": (C.c_char_p, [vp]),
        "olsgd_destroy": (i32, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _LIB = lib
    return lib


def _check(lib, status, ctx=None):
    if status != 0:
        raise OlsgdError(status, lib.olsgd_last_error(ctx).decode())


def _spec(kind, dims=(), gemm_bf16=0, flat_P=0):
    s = _ModelSpec()
    s.kind = _KINDS[kind]
    s.n_dims = len(dims)
    for i, d in enumerate(dims):
        s.dims[i] = int(d)
    s.gemm_bf16 = int(gemm_bf16)
    s.flat_P = int(flat_P)
    return s


def class_pairs(seed, m, device="cuda"):
    """olsgd_class_pairs: int32 tensor [m][2] on `device`."""
    lib = load_library()
    out = torch.empty((m, 2), dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream().cuda_stream
    _check(lib, lib.olsgd_class_pairs(int(seed), int(m), out.data_ptr(), stream))
    return out


def set_launch_overlap(on):
    """olsgd_set_launch_overlap: process-wide; returns the previous setting."""
    return bool(load_library().olsgd_set_launch_overlap(1 if on else 0))


def set_gemm_pairs(on):
    """olsgd_set_gemm_pairs: process-wide; returns the previous setting."""
    return bool(load_library().olsgd_set_gemm_pairs(1 if on else 0))


def tensor_core_launches():
    """olsgd_tensor_core_launches: launches of the tcgen05 kernels made by this process."""
    return int(load_library().olsgd_tensor_core_launches())


NOALLOC_MAX_WORKERS = 16384


def class_pairs_noalloc(seed, m, device="cpu"):
    """olsgd_class_pairs_noalloc: the same table, for callers that must not allocate
    (the library stages it in a fixed device array instead of fresh pinned memory).
    The output tensor here is still created by torch; pass your own memory to the C
    entry point if even that is not allowed."""
    lib = load_library()
    out = torch.empty((max(m, 0), 2), dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream().cuda_stream
    _check(lib, lib.olsgd_class_pairs_noalloc(int(seed), int(m), out.data_ptr(), stream))
    return out


class OverlapLocalSGD:
    """One olsgd context.  Method names mirror the C entry points."""

    def __init__(self, kind, *, m, tau, gamma, alpha, beta=0.0, mu=0.0, batch=1, seed=0,
                 dims=(), gemm_bf16=0, flat_P=0, x0, X=None, y=None, overlap=True,
                 local_sgd=False, worker_offset=0, m_total=0, epoch_sampling=False,
                 device="cuda"):
        self.lib = load_library()
        self.device = torch.device(device)
        self.spec = _spec(kind, dims, gemm_bf16, flat_P)
        self.hp = _HParams(int(m), int(tau), int(batch), 1 if local_sgd else 0, float(gamma), float(alpha),
                           float(beta), float(mu), int(seed), int(worker_offset), int(m_total),
                           1 if epoch_sampling else 0, 0)
        self.m, self.tau, self.batch, self.kind = int(m), int(tau), int(batch), kind
        P = C.c_int64()
        _check(self.lib, self.lib.olsgd_param_count(C.byref(self.spec), C.byref(P)))
        self.P = P.value
        nbytes = C.c_size_t()
        _check(self.lib, self.lib.olsgd_workspace_bytes(C.byref(self.spec), C.byref(self.hp),
                                                        C.byref(nbytes)))
        self.workspace_bytes = nbytes.value
        self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.main = torch.cuda.current_stream(self.device)
        self.side = torch.cuda.Stream(self.device) if overlap else self.main
        x0 = torch.as_tensor(x0, dtype=torch.float32).to(self.device).contiguous()
        assert x0.numel() == self.P, (x0.numel(), self.P)
        self._keep = [x0, X, y]
        data = None
        if kind != "flat":
            assert X.is_cuda and y.is_cuda and X.is_contiguous() and y.is_contiguous()
            assert X.dtype == torch.float32
            assert y.dtype == (torch.float32 if kind == "linreg" else torch.int32)
            data = _Data(X.data_ptr(), y.data_ptr(), X.shape[1])
        ctx = C.c_void_p()
        st = self.lib.olsgd_init(C.byref(ctx), C.byref(self.spec), C.byref(self.hp),
                                 C.byref(data) if data is not None else None, x0.data_ptr(),
                                 ws_ptr, nbytes.value, self.main.cuda_stream,
                                 self.side.cuda_stream)
        _check(self.lib, st)
        self.ctx = ctx

    # -- the C entry points ---------------------------------------------------
    def local_step(self, loss=None):
        _check(self.lib, self.lib.olsgd_local_step(self.ctx, loss.data_ptr() if loss is not None else None),
               self.ctx)

    def local_step_with_grads(self, g):
        assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()
        assert g.numel() == self.m * self.P
        _check(self.lib, self.lib.olsgd_local_step_with_grads(self.ctx, g.data_ptr()), self.ctx)

    def local_step_host(self, Xb, yb, loss=None):
        """Xb, yb (and loss) are HOST tensors, ideally pinned.  Xb is float32, or bfloat16 for
        a model whose GEMM operands are bf16 (olsgd_local_step_host_bf16)."""
        assert not Xb.is_cuda and not yb.is_cuda and Xb.is_contiguous() and yb.is_contiguous()
        assert Xb.dtype in (torch.float32, torch.bfloat16)
        assert Xb.numel() == self.m * self.batch * self.spec.dims[0]
        assert yb.numel() == self.m * self.batch and yb.element_size() == 4
        fn = (self.lib.olsgd_local_step_host if Xb.dtype == torch.float32
              else self.lib.olsgd_local_step_host_bf16)
        _check(self.lib, fn(self.ctx, Xb.data_ptr(), yb.data_ptr(),
                            loss.data_ptr() if loss is not None else None), self.ctx)

    def join(self):
        _check(self.lib, self.lib.olsgd_join(self.ctx), self.ctx)

    def selftest_wait_timeout(self, limit_ms):
        _check(self.lib, self.lib.olsgd_selftest_wait_timeout(self.ctx, int(limit_ms)), self.ctx)

    def clear_status(self):
        _check(self.lib, self.lib.olsgd_clear_status(self.ctx), self.ctx)

    def period_sync(self):
        _check(self.lib, self.lib.olsgd_period_sync(self.ctx), self.ctx)

    def set_anchor_fusion(self, on):
        _check(self.lib, self.lib.olsgd_set_anchor_fusion(self.ctx, 1 if on else 0), self.ctx)

    @property
    def anchor_fusion(self):
        return bool(self.lib.olsgd_anchor_fusion(self.ctx))

    @property
    def summed_floats(self):
        """Parameters of a row that the most recent anchor refresh took from partial sums
        formed by the sync step's own launches."""
        return int(self.lib.olsgd_summed_floats(self.ctx))

    def period_sync_begin(self, partial_sum):
        assert partial_sum.is_cuda and partial_sum.dtype == torch.float32
        assert partial_sum.numel() >= self.lib.olsgd_row_floats(self.ctx)
        _check(self.lib, self.lib.olsgd_period_sync_begin(self.ctx, partial_sum.data_ptr()), self.ctx)

    def period_sync_finish(self, total_sum):
        assert total_sum.is_cuda and total_sum.dtype == torch.float32
        _check(self.lib, self.lib.olsgd_period_sync_finish(self.ctx, total_sum.data_ptr()), self.ctx)

    def period_sync_sharded(self, buf, group=None):
        """Anchor refresh of a context that holds a shard of the workers: partial sum, all-reduce
        over `group` (torch.distributed, issued on the side stream), anchor update."""
        import torch.distributed as dist
        self.period_sync_begin(buf)
        with torch.cuda.stream(self.side):
            dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
        self.period_sync_finish(buf)

    def run(self, n_iters, loss=None):
        if loss is not None:
            assert loss.numel() >= n_iters * self.m and loss.dtype == torch.float32
        _check(self.lib, self.lib.olsgd_run(self.ctx, int(n_iters),
                                            loss.data_ptr() if loss is not None else None), self.ctx)

    def get_params(self, which, out=None):
        """which: 0..m-1 worker, -1 anchor z, -2 anchor momentum v, -3 virtual y,
        -4 mean model, -5-i local momentum u_i.  Returns a host float32 array unless
        `out` (host or device tensor) is given."""
        if out is None:
            out = torch.empty(self.P, dtype=torch.float32)
        _check(self.lib, self.lib.olsgd_get_params(self.ctx, int(which), out.data_ptr(), self.P),
               self.ctx)
        return out.numpy() if not out.is_cuda else out

    def set_params(self, which, src):
        src = torch.as_tensor(src, dtype=torch.float32).contiguous()
        assert src.numel() == self.P
        _check(self.lib, self.lib.olsgd_set_params(self.ctx, int(which), src.data_ptr(), self.P),
               self.ctx)

    def set_iteration(self, k):
        _check(self.lib, self.lib.olsgd_set_iteration(self.ctx, int(k)), self.ctx)

    def consensus_distance(self):
        out = C.c_double()
        _check(self.lib, self.lib.olsgd_consensus_distance(self.ctx, C.byref(out)), self.ctx)
        return out.value

    def get_indices(self, k):
        out = torch.empty((self.m, self.batch), dtype=torch.int32)
        _check(self.lib, self.lib.olsgd_get_indices(self.ctx, int(k), out.data_ptr()), self.ctx)
        return out.numpy()

    @property
    def iteration(self):
        return self.lib.olsgd_iteration(self.ctx)

    @property
    def launch_count(self):
        return self.lib.olsgd_launch_count(self.ctx)

    @property
    def graph_replays(self):
        return self.lib.olsgd_graph_replays(self.ctx)

    @property
    def graph_block(self):
        return self.lib.olsgd_graph_block(self.ctx)

    def profile_enable(self, on=True):
        _check(self.lib, self.lib.olsgd_profile_enable(self.ctx, 1 if on else 0), self.ctx)

    def profile_read(self, reset=True):
        n = len(KERNEL_CLASSES)
        launches = (C.c_int64 * n)()
        millis = (C.c_double * n)()
        _check(self.lib, self.lib.olsgd_profile_read(self.ctx, launches, millis, 1 if reset else 0),
               self.ctx)
        return {KERNEL_CLASSES[i]: (launches[i], millis[i]) for i in range(n)}

    def profile_read_layers(self, reset=True):
        """{class: [(launches, ms) per layer tag]} (olsgd_profile_read_layers)."""
        n = len(KERNEL_CLASSES) * MAX_DIMS
        launches = (C.c_int64 * n)()
        millis = (C.c_double * n)()
        _check(self.lib, self.lib.olsgd_profile_read_layers(self.ctx, launches, millis,
                                                            1 if reset else 0), self.ctx)
        return {KERNEL_CLASSES[i]: [(launches[i * MAX_DIMS + t], millis[i * MAX_DIMS + t])
                                    for t in range(MAX_DIMS)] for i in range(len(KERNEL_CLASSES))}

    # -- conveniences built from the calls above ---------------------------------
    def state(self):
        """Host copies: x [m][P], z [P], v [P]."""
        x = np.stack([self.get_params(i).copy() for i in range(self.m)])
        return x, self.get_params(-1).copy(), self.get_params(-2).copy()

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.olsgd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
