"""ctypes binding of libcdgrab.so: same names as ``include/cdgrab.h``, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  There is no CPU fallback: if the
shared library has not been built, or no sm_100 device is present, the calls raise.
PyTorch tensors are used as device buffers; their ``data_ptr()`` and the current CUDA stream
handle are what crosses the boundary.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# CDGRAB_LIB: file name (inside the package) of a diagnostic build to load instead
LIB_PATH = os.path.join(HERE, os.path.basename(os.environ.get("CDGRAB_LIB", "libcdgrab.so")))

F32, BF16 = 0, 1
OK = 0
ERR_INVALID, ERR_STATE, ERR_CUDA, ERR_NOMEM, ERR_NONFINITE, ERR_TIMEOUT, ERR_DEVICE = -1, -2, -3, -4, -5, -6, -7
ERR_TOO_LARGE = -8
ERR_CORRUPT = -9
PATH_AUTO, PATH_FUSED, PATH_FMA, PATH_UMMA = 0, 1, 2, 3
KERNEL_KINDS = ("gram", "combine", "scan", "update", "fused", "logreg")
PATH_NAMES = {PATH_FUSED: "fused", PATH_FMA: "fma", PATH_UMMA: "umma", 4: "independent", 5: "literal"}

# name -> (restype, argtypes); the single list of what include/cdgrab.h declares
SIGNATURES = {
    "cdgrab_create": (C.c_int, [C.c_int, C.c_int, C.c_longlong, C.c_int, C.POINTER(C.c_void_p)]),
    "cdgrab_create_independent": (C.c_int, [C.c_int, C.c_int, C.c_longlong, C.c_int, C.POINTER(C.c_void_p)]),
    "cdgrab_get_r_worker": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]),
    "cdgrab_create_shard": (C.c_int, [C.c_int, C.c_int, C.c_longlong, C.c_int, C.POINTER(C.c_void_p)]),
    "cdgrab_step_begin": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_step_finish": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_destroy": (C.c_int, [C.c_void_p]),
    "cdgrab_set_perms": (C.c_int, [C.c_void_p, C.c_void_p]),
    "cdgrab_begin_epoch": (C.c_int, [C.c_void_p, C.c_void_p]),
    "cdgrab_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_step_randomized": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_void_p]),
    "cdgrab_out_of_bound": (C.c_longlong, [C.c_void_p]),
    "cdgrab_step_randomized_seeded": (C.c_int, [C.c_void_p, C.c_void_p, C.c_ulonglong, C.c_uint, C.c_double, C.c_void_p]),
    "cdgrab_randomized_uniforms": (C.c_int, [C.c_ulonglong, C.c_uint, C.c_uint, C.c_int, C.c_void_p, C.c_void_p]),
    "cdgrab_step_mean": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_end_epoch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_get_signs": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_get_r": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_get_margins": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_get_perms": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_get_next_perms": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_status": (C.c_int, [C.c_void_p]),
    "cdgrab_clear_status": (C.c_int, [C.c_void_p]),
    "cdgrab_selftest_wait_timeout": (C.c_int, [C.c_void_p, C.c_longlong, C.POINTER(C.c_longlong)]),
    "cdgrab_state_bytes": (C.c_longlong, [C.c_void_p]),
    "cdgrab_save_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_longlong]),
    "cdgrab_load_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_longlong]),
    "cdgrab_path": (C.c_int, [C.c_void_p]),
    "cdgrab_launch_count": (C.c_longlong, [C.c_void_p]),
    "cdgrab_strerror": (C.c_char_p, [C.c_int]),
    "cdgrab_step_many": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "cdgrab_profile_enable": (C.c_int, [C.c_void_p, C.c_int]),
    "cdgrab_profile_read": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]),
    "cdgrab_logreg_grads": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_step_logreg": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_step_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cdgrab_herding_workspace_bytes": (C.c_longlong, [C.c_int, C.c_int, C.c_longlong]),
    "cdgrab_herding_objective": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_longlong, C.c_void_p,
                                           C.c_longlong, C.c_void_p, C.c_void_p]),
    "cdgrab_step_noalloc": (C.c_int, [C.c_int, C.c_longlong, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p]),
    "cdgrab_noalloc_status": (C.c_int, []),
}

_lib = None


class CdgrabError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().cdgrab_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{where}: {msg} ({code})")


def lib() -> C.CDLL:
    """Load libcdgrab.so (built in-tree by ``paper_2302_00845_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2302_00845_b200.build` "
                "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(code: int, where: str):
    if code != OK:
        raise CdgrabError(code, where)


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    """Raw pointer of a contiguous torch tensor or numpy array."""
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    assert t.flags["C_CONTIGUOUS"]
    return C.c_void_p(t.ctypes.data)


class CdGrab:
    """Order-server state for m workers x n items in R^d (see ``include/cdgrab.h``)."""

    def __init__(self, m: int, n: int, d: int, dtype: str | int = "f32", independent: bool = False,
                 shard: bool = False):
        code = {"f32": F32, "bf16": BF16}.get(dtype, dtype)
        h = C.c_void_p()
        if shard:         # one column shard of a coordinated order: d is the shard's width
            _check(lib().cdgrab_create_shard(m, n, d, code, C.byref(h)), "cdgrab_create_shard")
        elif independent:   # ID-GraB (PairBal): one running sum per worker
            _check(lib().cdgrab_create_independent(m, n, d, code, C.byref(h)), "cdgrab_create_independent")
        else:
            _check(lib().cdgrab_create(m, n, d, code, C.byref(h)), "cdgrab_create")
        self._h = h
        self.m, self.n, self.d, self.dtype = m, n, d, code

    # life cycle -------------------------------------------------------------------------
    def destroy(self):
        if getattr(self, "_h", None):
            lib().cdgrab_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    # the calls of the header ----------------------------------------------------------------
    def set_perms(self, perms):
        _check(lib().cdgrab_set_perms(self._h, _ptr(perms)), "cdgrab_set_perms")

    def begin_epoch(self, stream=None):
        _check(lib().cdgrab_begin_epoch(self._h, _stream_ptr(stream)), "cdgrab_begin_epoch")

    def step(self, grads, stream=None):
        """grads: CUDA tensor [2][m][d] of the handle's dtype."""
        _check(lib().cdgrab_step(self._h, _ptr(grads), _stream_ptr(stream)), "cdgrab_step")

    def step_randomized(self, grads, u, w: float, stream=None):
        """step() under the randomized rule: u CUDA float32 [m] uniforms, w > 0 the bound."""
        _check(lib().cdgrab_step_randomized(self._h, _ptr(grads), _ptr(u), float(w), _stream_ptr(stream)),
               "cdgrab_step_randomized")

    def step_randomized_seeded(self, grads, seed: int, epoch: int, w: float, stream=None):
        """step() under the randomized rule with the library's own counter-based draws."""
        _check(lib().cdgrab_step_randomized_seeded(self._h, _ptr(grads), int(seed), int(epoch), float(w),
                                                   _stream_ptr(stream)), "cdgrab_step_randomized_seeded")

    @property
    def out_of_bound(self) -> int:
        return int(lib().cdgrab_out_of_bound(self._h))

    def step_begin(self, grads, gram_out, stream=None):
        """Shard handle: pass 1; gram_out is a CUDA float64 tensor [m*m + m] for the partial (G, b)."""
        _check(lib().cdgrab_step_begin(self._h, _ptr(grads), _ptr(gram_out), _stream_ptr(stream)),
               "cdgrab_step_begin")

    def step_finish(self, grads, gram_in, stream=None):
        """Shard handle: decisions on the summed (G, b) and the update of this shard's slice of r."""
        _check(lib().cdgrab_step_finish(self._h, _ptr(grads), _ptr(gram_in), _stream_ptr(stream)),
               "cdgrab_step_finish")

    def step_mean(self, grads, mean_out, stream=None):
        """step() that also writes the average of each gather buffer into mean_out (CUDA float32 [2][d])."""
        _check(lib().cdgrab_step_mean(self._h, _ptr(grads), _ptr(mean_out), _stream_ptr(stream)),
               "cdgrab_step_mean")

    def step_many(self, grads, stream=None):
        """grads: contiguous CUDA tensor [count][2][m][d]; the count steps in one call."""
        _check(lib().cdgrab_step_many(self._h, _ptr(grads), int(grads.shape[0]), _stream_ptr(stream)),
               "cdgrab_step_many")

    def step_logreg(self, X, y, w, stream=None):
        """One balancing step straight from the feature rows (no gradient buffer)."""
        _check(lib().cdgrab_step_logreg(self._h, _ptr(X), _ptr(y), _ptr(w), _stream_ptr(stream)),
               "cdgrab_step_logreg")

    def step_host(self, grads_host, staging, stream=None):
        """grads_host: pinned host tensor [2][m][d]; staging: CUDA tensor of the same size."""
        _check(lib().cdgrab_step_host(self._h, _ptr(grads_host), _ptr(staging), _stream_ptr(stream)),
               "cdgrab_step_host")

    def end_epoch(self, perms_out=None, stream=None):
        p = _ptr(perms_out) if perms_out is not None else None
        _check(lib().cdgrab_end_epoch(self._h, p, _stream_ptr(stream)), "cdgrab_end_epoch")

    def logreg_grads(self, X, y, w, grads_out, stream=None):
        _check(lib().cdgrab_logreg_grads(self._h, _ptr(X), _ptr(y), _ptr(w), _ptr(grads_out),
                                         _stream_ptr(stream)), "cdgrab_logreg_grads")

    # read-back ------------------------------------------------------------------------------
    def _fetch(self, name, shape, dtype):
        import torch
        out = torch.empty(shape, dtype=dtype, device="cuda")
        _check(getattr(lib(), name)(self._h, _ptr(out), _stream_ptr()), name)
        torch.cuda.current_stream().synchronize()
        return out

    def signs(self):
        import torch
        return self._fetch("cdgrab_get_signs", (self.m, self.n // 2), torch.int8)

    def r(self):
        import torch
        return self._fetch("cdgrab_get_r", (self.d,), torch.float32)

    def r_worker(self, i: int):
        import torch
        out = torch.empty(self.d, dtype=torch.float32, device="cuda")
        _check(lib().cdgrab_get_r_worker(self._h, i, _ptr(out), _stream_ptr()), "cdgrab_get_r_worker")
        torch.cuda.current_stream().synchronize()
        return out

    def margins(self):
        import torch
        return self._fetch("cdgrab_get_margins", (self.m, self.n // 2), torch.float32)

    def perms(self):
        import torch
        return self._fetch("cdgrab_get_perms", (self.m, self.n), torch.int32)

    def next_perms(self):
        import torch
        return self._fetch("cdgrab_get_next_perms", (self.m, self.n), torch.int32)

    def save_state(self):
        """Host copy (numpy uint8 array) of everything needed to continue in another handle."""
        import numpy as np
        nbytes = int(lib().cdgrab_state_bytes(self._h))
        buf = np.empty(nbytes, dtype=np.uint8)
        _check(lib().cdgrab_save_state(self._h, buf.ctypes.data, nbytes), "cdgrab_save_state")
        return buf

    def load_state(self, buf):
        _check(lib().cdgrab_load_state(self._h, buf.ctypes.data, int(buf.nbytes)), "cdgrab_load_state")

    def status(self) -> int:
        return lib().cdgrab_status(self._h)

    def check_status(self):
        _check(self.status(), "cdgrab_status")

    def profile_enable(self, on: bool = True):
        _check(lib().cdgrab_profile_enable(self._h, int(on)), "cdgrab_profile_enable")

    def profile_read(self) -> dict:
        """{kernel kind: (total ms, launches)} for the launches recorded since profiling was enabled."""
        out = {}
        for kind, name in enumerate(KERNEL_KINDS):
            ms, cnt = C.c_double(), C.c_longlong()
            _check(lib().cdgrab_profile_read(self._h, kind, C.byref(ms), C.byref(cnt)), "cdgrab_profile_read")
            if cnt.value:
                out[name] = (ms.value, cnt.value)
        return out

    @property
    def path(self) -> str:
        return PATH_NAMES.get(lib().cdgrab_path(self._h), "?")

    @property
    def launch_count(self) -> int:
        return int(lib().cdgrab_launch_count(self._h))


def step_noalloc(grads, r, signs_out, stream=None):
    """cdgrab_step_noalloc on torch tensors: grads [2][m][d] (f32 or bf16), r float32 [d] updated in
    place, signs_out int8 [m].  Allocates nothing on the device."""
    import torch
    m, d = int(grads.shape[1]), int(grads.shape[2])
    code = F32 if grads.dtype == torch.float32 else BF16
    _check(lib().cdgrab_step_noalloc(m, d, code, _ptr(grads), _ptr(r), _ptr(signs_out), _stream_ptr(stream)),
           "cdgrab_step_noalloc")


def randomized_uniforms(seed: int, epoch: int, k: int, m: int, stream=None):
    """The m draws of (seed, epoch, k) as a CUDA float32 tensor."""
    import torch
    out = torch.empty(m, dtype=torch.float32, device="cuda")
    _check(lib().cdgrab_randomized_uniforms(int(seed), int(epoch), int(k), m, _ptr(out), _stream_ptr(stream)),
           "cdgrab_randomized_uniforms")
    return out


def noalloc_status() -> int:
    """cdgrab_noalloc_status: the device status of the step_noalloc calls so far (read and cleared)."""
    return int(lib().cdgrab_noalloc_status())


def herding_objective(z, perms, stream=None) -> float:
    """Eq. (7) on the device: z CUDA float32 [m][n][d] (by item id), perms CUDA int32 [m][n]."""
    import torch
    m, n, d = (int(v) for v in z.shape)
    nbytes = int(lib().cdgrab_herding_workspace_bytes(m, n, d))
    ws = torch.empty(nbytes // 8, dtype=torch.float64, device=z.device)
    out = torch.empty(1, dtype=torch.float64, device=z.device)
    _check(lib().cdgrab_herding_objective(_ptr(z), _ptr(perms), m, n, d, _ptr(ws), nbytes, _ptr(out),
                                          _stream_ptr(stream)), "cdgrab_herding_objective")
    return float(out.item())


class ShardedCdGrab:
    """One rank of a column-sharded order server over ``torch.distributed``: this rank owns
    d_local columns; every step all-reduces m*m + m doubles (NCCL on GPUs)."""

    def __init__(self, m: int, n: int, d_local: int, dtype="f32", group=None):
        self.group = group
        self._attach(CdGrab(m, n, d_local, dtype, shard=True), m, "cuda")

    def _attach(self, handle, m: int, device):
        """The shard handle this rank drives and the buffer its partial (G, b) is exchanged in."""
        import torch
        self.h = handle
        self.gram = torch.empty(m * m + m, dtype=torch.float64, device=device)

    def begin_epoch(self):
        self.h.begin_epoch()

    def step(self, grads_local):
        import torch.distributed as dist
        self.h.step_begin(grads_local, self.gram)
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1:
            dist.all_reduce(self.gram, op=dist.ReduceOp.SUM, group=self.group)
        self.h.step_finish(grads_local, self.gram)

    def end_epoch(self, perms_out=None):
        self.h.end_epoch(perms_out)

    def destroy(self):
        self.h.destroy()
