"""ctypes binding of libst3.so: argument marshalling only, one Python function per C entry point.

Every step of the method runs inside the library's CUDA kernels; torch is used by callers for
device memory and streams, never for the computation.  There is no CPU fallback: if the shared
library is missing or does not load, `load()` raises.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libst3.so")

ST3_OK = 0
STATUS_NAMES = ["ST3_OK", "ST3_ERR_INVALID_ARG", "ST3_ERR_WORKSPACE_TOO_SMALL", "ST3_ERR_BAD_STATE",
                "ST3_ERR_CAPACITY", "ST3_ERR_CUDA", "ST3_ERR_DEVICE_CHECK", "ST3_ERR_UNSUPPORTED"]
ST3_F32, ST3_BF16 = 0, 1
ST3_ANNEAL_COSINE, ST3_ANNEAL_NONE, ST3_ANNEAL_LINEAR, ST3_ANNEAL_EXP = 0, 1, 2, 3
DEV_COUNT_MISMATCH, DEV_NONFINITE, DEV_COPY_TIMEOUT, DEV_RANGE = 1, 2, 4, 8

EXPORTS = ["st3_schedule_count", "st3_workspace_size", "st3_create", "st3_prefill_select",
           "st3_prefill_select_scored", "st3_decode_step",
           "st3_decode_step_host", "st3_prefill_select_host", "st3_host_sync", "st3_get_kept", "st3_get_rows", "st3_get_status", "st3_rows_held",
           "st3_set_overlap", "st3_profile_enable", "st3_profile_read", "st3_launch_count", "st3_status_string", "st3_destroy",
           "st3_attend_noalloc", "st3_prefill_attend", "st3_prefill_attend_kept"]


class Config(C.Structure):
    """Mirror of `st3_config` (include/st3.h)."""
    _fields_ = [(n, C.c_int32) for n in (
        "num_layers", "num_heads", "head_dim", "dtype", "batch", "sys_len", "num_visual", "max_text_len",
        "max_decode_steps", "first_prune_layer", "stride", "first_ratio_bp", "step_ratio_bp", "anneal",
        "disable_trim", "rows_per_chunk", "static_rank", "stage_shared", "host_prefill")] + [("lazy_mask", C.c_uint64), ("tau", C.c_double), ("sigma", C.c_double)]


class St3Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where}: {name}")


_lib = None


def load():
    """Loads libst3.so (once) and declares the prototypes.  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_2412_20105_b200.build); "
                           "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    cfgp = C.POINTER(Config)
    lib.st3_schedule_count.argtypes = [cfgp, i32, i32]
    lib.st3_schedule_count.restype = i32
    lib.st3_workspace_size.argtypes = [cfgp, C.POINTER(C.c_size_t)]
    lib.st3_create.argtypes = [cfgp, vp, C.c_size_t, C.POINTER(vp)]
    lib.st3_prefill_select.argtypes = [vp, i32, i32, vp, vp, vp, C.POINTER(i32), vp, vp]
    lib.st3_prefill_select_scored.argtypes = [vp, i32, i32, vp, vp, vp, C.POINTER(i32), vp, vp, vp]
    lib.st3_decode_step.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.st3_decode_step_host.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.st3_prefill_select_host.argtypes = [vp, i32, i32, vp, vp, vp, C.POINTER(i32), vp, vp]
    lib.st3_host_sync.argtypes = [vp, vp]
    lib.st3_get_kept.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.st3_get_rows.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.st3_get_status.argtypes = [vp, C.POINTER(i32)]
    lib.st3_rows_held.argtypes = [vp, C.POINTER(i64), C.POINTER(i64)]
    lib.st3_set_overlap.argtypes = [vp, i32]
    lib.st3_profile_enable.argtypes = [vp, i32]
    lib.st3_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(i64),
                                     C.POINTER(i64)]
    lib.st3_launch_count.argtypes = [vp]
    lib.st3_launch_count.restype = i64
    lib.st3_status_string.argtypes = [C.c_int]
    lib.st3_status_string.restype = C.c_char_p
    lib.st3_destroy.argtypes = [vp]
    lib.st3_attend_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.st3_prefill_attend.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.st3_prefill_attend_kept.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, i32, vp]
    for name in EXPORTS:
        if name not in ("st3_schedule_count", "st3_launch_count", "st3_status_string"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _check(code: int, where: str):
    if code != ST3_OK:
        raise St3Error(code, where)


def make_config(*, num_layers, num_heads, head_dim, dtype, batch, sys_len, num_visual, max_text_len,
                max_decode_steps, stride, step_ratio_bp, tau, first_prune_layer=3, first_ratio_bp=5000,
                anneal=ST3_ANNEAL_COSINE, disable_trim=0, rows_per_chunk=0, sigma=20.0, static_rank=0, stage_shared=0, lazy_mask=0,
                host_prefill=0) -> Config:
    dt = {"f32": ST3_F32, "bf16": ST3_BF16}.get(dtype, dtype)
    return Config(num_layers, num_heads, head_dim, dt, batch, sys_len, num_visual, max_text_len,
                  max_decode_steps, first_prune_layer, stride, first_ratio_bp, step_ratio_bp, anneal,
                  int(disable_trim), rows_per_chunk, int(static_rank), int(stage_shared), int(host_prefill), int(lazy_mask),
                  float(tau), float(sigma))


def st3_schedule_count(cfg: Config, layer: int, step: int) -> int:
    return load().st3_schedule_count(C.byref(cfg), layer, step)


def st3_workspace_size(cfg: Config) -> int:
    n = C.c_size_t(0)
    _check(load().st3_workspace_size(C.byref(cfg), C.byref(n)), "st3_workspace_size")
    return n.value


def st3_create(cfg: Config, workspace_ptr: int, nbytes: int) -> int:
    h = C.c_void_p(None)
    _check(load().st3_create(C.byref(cfg), workspace_ptr, nbytes, C.byref(h)), "st3_create")
    return h.value


def st3_prefill_select(ctx, layer_begin, layer_count, q_last, k, v, text_len, out, stream=0):
    """q_last/k/v/out are device addresses (ints); text_len is a host sequence of ints."""
    arr = (C.c_int32 * len(text_len))(*[int(x) for x in text_len])
    _check(load().st3_prefill_select(ctx, layer_begin, layer_count, q_last, k, v, arr, out, stream),
           "st3_prefill_select")


def st3_prefill_select_scored(ctx, layer_begin, layer_count, q_last, k, v, text_len, scores, out, stream=0):
    """As st3_prefill_select, but the kept set comes from `scores` (device address, fp32
    [layer_count][B][num_visual]) and the layer attends over the kept rows only."""
    arr = (C.c_int32 * len(text_len))(*[int(x) for x in text_len])
    _check(load().st3_prefill_select_scored(ctx, layer_begin, layer_count, q_last, k, v, arr, scores, out, stream),
           "st3_prefill_select_scored")


def st3_decode_step(ctx, step, layer_begin, layer_count, q, k_new, v_new, out, stream=0):
    _check(load().st3_decode_step(ctx, step, layer_begin, layer_count, q, k_new, v_new, out, stream),
           "st3_decode_step")


def st3_decode_step_host(ctx, step, layer_begin, layer_count, q, k_new, v_new, out, stream=0):
    _check(load().st3_decode_step_host(ctx, step, layer_begin, layer_count, q, k_new, v_new, out, stream),
           "st3_decode_step_host")


def st3_prefill_select_host(ctx, layer_begin, layer_count, q_last, k, v, text_len, out, stream=0):
    """As st3_prefill_select with pinned HOST addresses; needs a config with host_prefill=1."""
    arr = (C.c_int32 * len(text_len))(*[int(x) for x in text_len])
    _check(load().st3_prefill_select_host(ctx, layer_begin, layer_count, q_last, k, v, arr, out, stream),
           "st3_prefill_select_host")


def st3_host_sync(ctx, stream=0):
    _check(load().st3_host_sync(ctx, stream), "st3_host_sync")


def st3_get_kept(ctx, layer, ids, count, mass=None, stream=0):
    _check(load().st3_get_kept(ctx, layer, ids, count, mass, stream), "st3_get_kept")


def st3_get_rows(ctx, layer, b, h, k_vis=None, v_vis=None, k_txt=None, v_txt=None, stream=0):
    _check(load().st3_get_rows(ctx, layer, b, h, k_vis, v_vis, k_txt, v_txt, stream), "st3_get_rows")


def st3_get_status(ctx, raise_on_error=True) -> int:
    w = C.c_int32(0)
    code = load().st3_get_status(ctx, C.byref(w))
    if raise_on_error and code != ST3_OK:
        raise St3Error(code, f"st3_get_status (device word {w.value})")
    return w.value


def st3_rows_held(ctx):
    a, b = C.c_int64(0), C.c_int64(0)
    _check(load().st3_rows_held(ctx, C.byref(a), C.byref(b)), "st3_rows_held")
    return a.value, b.value


def st3_set_overlap(ctx, on: bool):
    _check(load().st3_set_overlap(ctx, int(on)), "st3_set_overlap")


def st3_profile_enable(ctx, on: bool):
    _check(load().st3_profile_enable(ctx, int(on)), "st3_profile_enable")


def st3_profile_read(ctx):
    a, f = C.c_double(0), C.c_double(0)
    na, nf = C.c_int64(0), C.c_int64(0)
    _check(load().st3_profile_read(ctx, C.byref(a), C.byref(f), C.byref(na), C.byref(nf)), "st3_profile_read")
    return a.value, f.value, na.value, nf.value


def st3_launch_count(ctx) -> int:
    return load().st3_launch_count(ctx)


def st3_status_string(code: int) -> str:
    return load().st3_status_string(code).decode()


def st3_destroy(ctx):
    _check(load().st3_destroy(ctx), "st3_destroy")


def st3_prefill_attend(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len, head_dim, dtype,
                       sys_len, num_visual, stream=0):
    """Causal attention of a whole prompt on the tensor cores (device addresses; see st3.h)."""
    dt = {"f32": ST3_F32, "bf16": ST3_BF16}.get(dtype, dtype)
    _check(load().st3_prefill_attend(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len,
                                     head_dim, dt, sys_len, num_visual, stream), "st3_prefill_attend")


def st3_prefill_attend_kept(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len, head_dim,
                            dtype, sys_len, num_visual, ids, num_visual_total, stream=0):
    """The same for a prompt that holds only the visual tokens `ids` names; scores come out by original index."""
    dt = {"f32": ST3_F32, "bf16": ST3_BF16}.get(dtype, dtype)
    _check(load().st3_prefill_attend_kept(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len,
                                          head_dim, dt, sys_len, num_visual, ids, num_visual_total, stream),
           "st3_prefill_attend_kept")


def st3_attend_noalloc(q, k, v, out, num_heads, num_rows, head_dim, dtype, stream=0):
    """Workspace-free attention for callers that may not allocate device memory: q/k/v/out are
    device addresses, the split partials live in a fixed array inside the library (see st3.h for
    the size limit and the sharing rules)."""
    dt = {"f32": ST3_F32, "bf16": ST3_BF16}.get(dtype, dtype)
    _check(load().st3_attend_noalloc(q, k, v, out, num_heads, num_rows, head_dim, dt, stream), "st3_attend_noalloc")


class Context:
    """Owns a torch-allocated workspace and a library context; forwards to the C entry points.

    Torch supplies device memory and the current stream only.  Tensors passed in must be CUDA,
    contiguous and of the configured dtype.
    """

    def __init__(self, cfg: Config, device="cuda:0"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        load()
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device(device)
        self.dtype = torch.bfloat16 if cfg.dtype == ST3_BF16 else torch.float32
        nbytes = st3_workspace_size(cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            self.handle = st3_create(cfg, self._ws_ptr, nbytes)
        self.workspace_bytes = nbytes

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def _ptr(self, t):
        assert t.is_cuda and t.is_contiguous() and t.dtype == self.dtype, (t.device, t.dtype, t.is_contiguous())
        return t.data_ptr()

    def io_shape(self, layer_count=None):
        c = self.cfg
        return (c.num_layers if layer_count is None else layer_count, c.batch, c.num_heads, c.head_dim)

    def prefill_select(self, q_last, k, v, text_len, out, layer_begin=0):
        st3_prefill_select(self.handle, layer_begin, q_last.shape[0], self._ptr(q_last), self._ptr(k), self._ptr(v),
                           text_len, self._ptr(out), self._stream())

    def prefill_select_scored(self, q_last, k, v, text_len, scores, out, layer_begin=0):
        assert scores.is_cuda and scores.is_contiguous() and scores.dtype == self.torch.float32
        st3_prefill_select_scored(self.handle, layer_begin, q_last.shape[0], self._ptr(q_last), self._ptr(k),
                                  self._ptr(v), text_len, scores.data_ptr(), self._ptr(out), self._stream())

    def decode_step(self, step, q, k_new, v_new, out, layer_begin=0):
        st3_decode_step(self.handle, step, layer_begin, q.shape[0], self._ptr(q), self._ptr(k_new), self._ptr(v_new),
                        self._ptr(out), self._stream())

    def decode_step_host(self, step, q, k_new, v_new, out, layer_begin=0):
        """q/k_new/v_new/out are pinned HOST tensors."""
        st3_decode_step_host(self.handle, step, layer_begin, q.shape[0], q.data_ptr(), k_new.data_ptr(),
                             v_new.data_ptr(), out.data_ptr(), self._stream())

    def prefill_select_host(self, q_last, k, v, text_len, out, layer_begin=0):
        """q_last/k/v/out are pinned HOST tensors."""
        st3_prefill_select_host(self.handle, layer_begin, q_last.shape[0], q_last.data_ptr(), k.data_ptr(),
                                v.data_ptr(), text_len, out.data_ptr(), self._stream())

    def host_sync(self):
        st3_host_sync(self.handle, self._stream())

    def get_kept(self, layer, with_mass=True):
        t, c = self.torch, self.cfg
        ids = t.empty((c.batch, max(1, c.num_visual)), dtype=t.int32, device=self.device)
        cnt = t.empty((c.batch,), dtype=t.int32, device=self.device)
        mass = t.empty((c.batch, max(1, c.num_visual)), dtype=t.float32, device=self.device) if with_mass else None
        st3_get_kept(self.handle, layer, ids.data_ptr(), cnt.data_ptr(), mass.data_ptr() if with_mass else None,
                     self._stream())
        return ids, cnt, mass

    def get_rows(self, layer, b, h):
        t, c = self.torch, self.cfg
        cap = c.sys_len + c.max_text_len + c.max_decode_steps
        kv = [t.empty((max(1, c.num_visual), c.head_dim), dtype=self.dtype, device=self.device) for _ in range(2)]
        tx = [t.empty((cap, c.head_dim), dtype=self.dtype, device=self.device) for _ in range(2)]
        st3_get_rows(self.handle, layer, b, h, kv[0].data_ptr(), kv[1].data_ptr(), tx[0].data_ptr(), tx[1].data_ptr(),
                     self._stream())
        return kv[0], kv[1], tx[0], tx[1]

    def status(self, raise_on_error=True):
        return st3_get_status(self.handle, raise_on_error)

    def rows_held(self):
        return st3_rows_held(self.handle)

    def launch_count(self):
        return st3_launch_count(self.handle)

    def close(self):
        if self.handle:
            self.torch.cuda.synchronize(self.device)
            st3_destroy(self.handle)
            self.handle = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def config_from_workload(wl, **overrides) -> Config:
    """Config for one of the synthetic workloads (any object with the Workload fields)."""
    kw = dict(num_layers=wl.num_layers, num_heads=wl.num_heads, head_dim=wl.head_dim, dtype=wl.dtype,
              batch=wl.batch, sys_len=wl.sys_len, num_visual=wl.num_visual, max_text_len=wl.text_len_max,
              max_decode_steps=wl.decode_steps, stride=wl.stride, step_ratio_bp=wl.step_ratio_bp, tau=wl.tau,
              first_prune_layer=wl.first_prune_layer, first_ratio_bp=wl.first_ratio_bp)
    kw.update(overrides)
    return make_config(**kw)
