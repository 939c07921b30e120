"""Thin ctypes binding of libvattn (argument marshalling only; all computation is in the CUDA kernels).

Same names as the C ABI (include/vattn.h).  PyTorch supplies device memory and streams, nothing else.
Loading fails loudly when the library has not been built: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvattn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA = 0, -1, -2, -3, -4
DTYPE_FP32, DTYPE_BF16 = 0, 1
STATUS_BAD_BLOCK, STATUS_BAD_SEQLEN, STATUS_BAND_OVERFLOW, STATUS_NONFINITE, STATUS_WAIT_TIMEOUT = 1, 2, 4, 8, 16

EXPORTS = ["vattn_plan_create", "vattn_plan_destroy", "vattn_workspace_bytes", "vattn_set_workspace",
           "vattn_set_params", "vattn_set_debug", "vattn_decode", "vattn_dense_decode",
           "vattn_host_staging_bytes", "vattn_decode_host", "vattn_last_status", "vattn_last_launch_count",
           "vattn_strerror", "vattn_normal_quantile", "vattn_set_profiling", "vattn_read_profile",
           "vattn_dense_decode_noalloc", "vattn_set_stop_after", "vattn_probe_bounded_wait", "vattn_noalloc_last_status"]
NOALLOC_SCRATCH_BYTES = 4 << 20
KERNEL_NAMES = ["k_score", "k_walk", "k_select", "k_stats", "k_gather"]
NUM_TICKS = 8
# measurement builds (VATTN_DEFINES="VATTN_PHASE_TICKS") stamp phases inside the kernels into further rows
TICK_ROWS = 2560 if "VATTN_PHASE_TICKS" in os.environ.get("VATTN_DEFINES", "") else NUM_TICKS
TICK_NAMES = ["k_zero", "k_score", "k_walk", "k_select", "k_stats", "k_gather", "topk", "budget"]


class Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("block_size", C.c_int32), ("max_blocks_per_seq", C.c_int32),
                ("num_blocks", C.c_int32), ("max_seq_len", C.c_int32), ("dtype", C.c_int32),
                ("kv_stride_block", C.c_int64), ("kv_stride_head", C.c_int64), ("kv_stride_token", C.c_int64),
                ("q_len", C.c_int32)]


class Params(C.Structure):
    _fields_ = [("base_rate", C.c_float), ("topk_frac", C.c_float), ("scale", C.c_float), ("mode", C.c_int32),
                ("layer", C.c_int32), ("step", C.c_int32), ("rng_head_is_kv", C.c_int32),
                ("force_budget", C.c_int32), ("force_budget_on", C.c_int32), ("gather_mode", C.c_int32),
                ("nested_base", C.c_int32)]


class Debug(C.Structure):
    _fields_ = [("topk_idx", C.c_void_p), ("topk_cnt", C.c_void_p), ("base_idx", C.c_void_p),
                ("base_cnt", C.c_void_p), ("dyn_idx", C.c_void_p), ("dyn_cnt", C.c_void_p),
                ("budgets", C.c_void_p), ("stats", C.c_void_p), ("scores", C.c_void_p), ("paths", C.c_void_p),
                ("kernel_ticks", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it is missing (build it with `python -m paper_2510_05688_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA library first "
                           "(python -m paper_2510_05688_b200.build); there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, u64, f32, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_float, C.c_size_t
    L.vattn_plan_create.argtypes = [C.POINTER(Shape), C.POINTER(vp)]
    L.vattn_plan_create.restype = i32
    L.vattn_plan_destroy.argtypes = [vp]
    L.vattn_plan_destroy.restype = None
    L.vattn_workspace_bytes.argtypes = [vp]
    L.vattn_workspace_bytes.restype = sz
    L.vattn_set_workspace.argtypes = [vp, vp, sz]
    L.vattn_set_workspace.restype = i32
    L.vattn_set_params.argtypes = [vp, C.POINTER(Params)]
    L.vattn_set_params.restype = i32
    L.vattn_set_debug.argtypes = [vp, C.POINTER(Debug)]
    L.vattn_set_debug.restype = i32
    L.vattn_decode.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, f32, u64, vp, vp]
    L.vattn_decode.restype = i32
    L.vattn_dense_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.vattn_dense_decode.restype = i32
    L.vattn_host_staging_bytes.argtypes = [vp]
    L.vattn_host_staging_bytes.restype = sz
    L.vattn_decode_host.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, f32, u64, vp, vp, vp]
    L.vattn_decode_host.restype = i32
    L.vattn_last_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    L.vattn_last_status.restype = i32
    L.vattn_noalloc_last_status.argtypes = [C.POINTER(C.c_uint32), vp]
    L.vattn_noalloc_last_status.restype = i32
    L.vattn_probe_bounded_wait.argtypes = [vp, C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), vp]
    L.vattn_probe_bounded_wait.restype = i32
    L.vattn_last_launch_count.argtypes = [vp]
    L.vattn_last_launch_count.restype = i32
    L.vattn_strerror.argtypes = [i32]
    L.vattn_strerror.restype = C.c_char_p
    L.vattn_set_stop_after.argtypes = [vp, i32]
    L.vattn_set_stop_after.restype = i32
    L.vattn_set_profiling.argtypes = [vp, i32]
    L.vattn_set_profiling.restype = i32
    L.vattn_read_profile.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int)]
    L.vattn_read_profile.restype = i32
    L.vattn_dense_decode_noalloc.argtypes = [C.POINTER(Shape), f32, vp, vp, vp, vp, vp, vp, vp]
    L.vattn_dense_decode_noalloc.restype = i32
    L.vattn_normal_quantile.argtypes = [C.c_double]
    L.vattn_normal_quantile.restype = C.c_double
    _lib = L
    return L


class VattnError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().vattn_strerror(code).decode()} ({code})")


def _check(code, where):
    if code != OK:
        raise VattnError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Plan:
    """Owner of one vattn_plan plus the torch tensors backing its workspace and debug buffers."""

    def __init__(self, *, batch, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq, num_blocks, max_seq_len,
                 dtype, block_size=16, kv_strides=(0, 0, 0), q_len=1, device="cuda", alloc_workspace=True):
        self.shape = Shape(batch, num_q_heads, num_kv_heads, head_dim, block_size, max_blocks_per_seq, num_blocks,
                           max_seq_len, dtype, *kv_strides, q_len)
        h = C.c_void_p()
        _check(lib().vattn_plan_create(C.byref(self.shape), C.byref(h)), "vattn_plan_create")
        self._h = h
        self.device = device
        self.workspace = None
        self.debug = None
        self._staging = None
        if alloc_workspace:
            import torch
            nbytes = self.workspace_bytes()
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
            self.set_workspace(self.workspace.data_ptr(), nbytes)

    def __del__(self):
        h = getattr(self, "_h", None)
        if h is not None and h.value and _lib is not None:      # module globals are gone at interpreter exit
            _lib.vattn_plan_destroy(h)
            self._h = None

    # -- direct ABI calls
    def workspace_bytes(self) -> int:
        return int(lib().vattn_workspace_bytes(self._h))

    def set_workspace(self, ptr, nbytes):
        _check(lib().vattn_set_workspace(self._h, C.c_void_p(ptr), nbytes), "vattn_set_workspace")

    def set_params(self, **kw):
        p = Params()
        p.force_budget = -1
        fb = kw.pop("force_budget", None)
        if fb is not None and fb >= 0:
            p.force_budget, p.force_budget_on = int(fb), 1
        for k_, v in kw.items():
            if v is not None:
                setattr(p, k_, v)
        _check(lib().vattn_set_params(self._h, C.byref(p)), "vattn_set_params")

    def enable_debug(self):
        """Allocate device buffers for every introspection output and register them."""
        import torch
        s = self.shape
        # with q_len > 1 the head axis is [KV head, query token, head within the group] flattened
        BH, cap = (s.batch, s.num_q_heads * max(1, s.q_len)), s.max_seq_len
        dev = self.device
        i32 = torch.int32
        self.debug = dict(
            topk_idx=torch.zeros(*BH, cap, dtype=i32, device=dev), topk_cnt=torch.zeros(*BH, dtype=i32, device=dev),
            base_idx=torch.zeros(*BH, cap, dtype=i32, device=dev), base_cnt=torch.zeros(*BH, dtype=i32, device=dev),
            dyn_idx=torch.zeros(*BH, cap, dtype=i32, device=dev), dyn_cnt=torch.zeros(*BH, dtype=i32, device=dev),
            budgets=torch.zeros(*BH, 4, dtype=i32, device=dev),
            stats=torch.zeros(*BH, 8, dtype=torch.float64, device=dev),
            scores=torch.zeros(*BH, cap, dtype=torch.float32, device=dev),
            paths=torch.zeros(*BH, dtype=i32, device=dev))
        d = Debug(**{k_: v.data_ptr() for k_, v in self.debug.items()})
        _check(lib().vattn_set_debug(self._h, C.byref(d)), "vattn_set_debug")
        return self.debug

    def disable_debug(self):
        _check(lib().vattn_set_debug(self._h, None), "vattn_set_debug")
        self.debug = None

    def enable_kernel_ticks(self):
        """Register only the device-side time-stamp buffer ([NUM_TICKS, 2] int64, rows named by TICK_NAMES).
        Call reset_kernel_ticks() before the step to observe, read the tensor after it."""
        import torch
        self.ticks = torch.zeros(TICK_ROWS, 2, dtype=torch.int64, device=self.device)
        d = Debug(kernel_ticks=self.ticks.data_ptr())
        _check(lib().vattn_set_debug(self._h, C.byref(d)), "vattn_set_debug")
        self.reset_kernel_ticks()
        return self.ticks

    def reset_kernel_ticks(self):
        self.ticks[:, 0] = -1          # all ones: the largest unsigned value, for the atomic minimum
        self.ticks[:, 1] = 0

    def decode(self, q, k_cache, v_cache, block_table, seq_lens, sink, window, k, eps, delta, seed, out, stream=None):
        _check(lib().vattn_decode(self._h, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                                  int(sink), int(window), int(k), float(eps), float(delta), int(seed), _ptr(out),
                                  C.c_void_p(_stream(stream))), "vattn_decode")
        return out

    def dense_decode(self, q, k_cache, v_cache, block_table, seq_lens, out, stream=None):
        _check(lib().vattn_dense_decode(self._h, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                        _ptr(seq_lens), _ptr(out), C.c_void_p(_stream(stream))), "vattn_dense_decode")
        return out

    def decode_host(self, q_host, k_cache, v_cache, block_table_host, seq_lens_host, sink, window, k, eps, delta, seed,
                    out_host, stream=None):
        """q / block_table / seq_lens / out are HOST (ideally pinned) tensors; the caches stay on the device."""
        import torch
        if self._staging is None:
            self._staging = torch.empty(int(lib().vattn_host_staging_bytes(self._h)), dtype=torch.uint8,
                                        device=self.device)
        _check(lib().vattn_decode_host(self._h, _ptr(q_host), _ptr(k_cache), _ptr(v_cache), _ptr(block_table_host),
                                       _ptr(seq_lens_host), int(sink), int(window), int(k), float(eps), float(delta),
                                       int(seed), _ptr(out_host), _ptr(self._staging), C.c_void_p(_stream(stream))),
               "vattn_decode_host")
        return out_host

    def last_status(self, stream=None) -> int:
        bits = C.c_uint32(0)
        _check(lib().vattn_last_status(self._h, C.c_void_p(_stream(stream)), C.byref(bits)), "vattn_last_status")
        return int(bits.value)

    def set_stop_after(self, kernels: int):
        """Measurement aid: decode() enqueues only its first `kernels` kernels (0 = the whole step)."""
        _check(lib().vattn_set_stop_after(self._h, int(kernels)), "vattn_set_stop_after")

    def set_profiling(self, enable: bool):
        _check(lib().vattn_set_profiling(self._h, 1 if enable else 0), "vattn_set_profiling")

    def read_profile(self):
        """(dict kernel name -> summed ms, calls) since profiling was enabled or last read."""
        ms = (C.c_float * len(KERNEL_NAMES))()
        calls = C.c_int(0)
        _check(lib().vattn_read_profile(self._h, ms, C.byref(calls)), "vattn_read_profile")
        return {n: float(ms[i]) for i, n in enumerate(KERNEL_NAMES)}, int(calls.value)

    def probe_bounded_wait(self, spins: int, stream=None):
        """Run the bounded wait primitive alone on a word that nothing publishes: (ran_out, waited_us)."""
        ran, us = C.c_uint32(0), C.c_uint32(0)
        _check(lib().vattn_probe_bounded_wait(self._h, C.c_uint32(int(spins)), C.byref(ran), C.byref(us),
                                              C.c_void_p(_stream(stream))), "vattn_probe_bounded_wait")
        return int(ran.value), int(us.value)

    def last_launch_count(self) -> int:
        return int(lib().vattn_last_launch_count(self._h))


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


def dense_decode_noalloc(shape: Shape, q, k_cache, v_cache, block_table, seq_lens, out, scale=0.0, stream=None):
    """Dense decode through the entry point that needs no plan and no workspace: for callers that
    cannot allocate device memory (everything handed to a cache pool, or cudaMalloc off limits on
    their path).  Returns the ABI's return code instead of raising, so callers can test the limits."""
    return int(lib().vattn_dense_decode_noalloc(C.byref(shape), float(scale), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                                _ptr(block_table), _ptr(seq_lens), _ptr(out),
                                                C.c_void_p(_stream(stream))))


def noalloc_last_status(stream=None) -> int:
    """Status bits of the last dense_decode_noalloc call on the current device (waits for the stream)."""
    bits = C.c_uint32(0)
    _check(lib().vattn_noalloc_last_status(C.byref(bits), C.c_void_p(_stream(stream))), "vattn_noalloc_last_status")
    return int(bits.value)


def normal_quantile(x: float) -> float:
    return float(lib().vattn_normal_quantile(float(x)))


# ----------------------------------------------------------------------------- convenience for tests / bench
def case_to_device(case, device="cuda"):
    """Upload a synth.Case; bf16 arrays travel as their bit patterns and are viewed as torch.bfloat16."""
    import numpy as np
    import torch

    def up(a):
        if case.dtype == "bf16":
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)

    return dict(q=up(case.q), k_cache=up(case.k_cache), v_cache=up(case.v_cache),
                block_table=torch.from_numpy(case.block_table).to(device),
                seq_lens=torch.from_numpy(case.seq_lens).to(device))


def plan_for_case(case, device="cuda", max_seq_len=None, q_len=1) -> Plan:
    msl = int(max_seq_len if max_seq_len is not None else case.max_blocks_per_seq * 16)
    return Plan(batch=case.batch, num_q_heads=case.num_q_heads, num_kv_heads=case.num_kv_heads,
                head_dim=case.head_dim, max_blocks_per_seq=case.max_blocks_per_seq, num_blocks=case.num_blocks,
                max_seq_len=msl, dtype=DTYPE_BF16 if case.dtype == "bf16" else DTYPE_FP32, q_len=q_len, device=device)
