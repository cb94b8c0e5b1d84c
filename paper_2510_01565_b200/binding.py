"""ctypes binding of libdit.so: argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; torch is used
here for device memory and streams.  Loading fails loudly when the library has
not been built (there is no CPU or eager fallback).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdit.so")

DIT_OK = 0
DIT_FLAG_QK_RMSNORM = 1
DIT_FLAG_ROPE_2D = 2
DIT_FLAG_FP8_GEMM = 4
DIT_FLAG_BF16_OPERANDS = 8
STATUS_NAMES = ["DIT_OK", "DIT_ERR_INVALID_ARG", "DIT_ERR_SHAPE", "DIT_ERR_CAPACITY", "DIT_ERR_NOT_LOADED",
                "DIT_ERR_UNSUPPORTED_ARCH", "DIT_ERR_CUDA", "DIT_ERR_TIMEOUT", "DIT_ERR_INTERNAL"]
KERNEL_KINDS = ["modulation", "ln_modulate", "gemm_qkv", "attention", "gemm_proj", "gemm_fc1", "gemm_fc2", "quantize"]
TAPS = {"h": 0, "qkv": 1, "attn": 2, "u": 3, "mod": 4, "stream": 5}

EXPORTS = ["dit_workspace_bytes", "dit_ctx_create", "dit_ctx_destroy", "dit_load_block_weights", "dit_load_parallel_block_weights", "dit_load_dual_block_weights",
           "dit_pack_requests", "dit_pack_tokens", "dit_step_forward", "dit_step_forward_requests", "dit_step_forward_host", "dit_step_forward_host_async", "dit_host_wait",
           "dit_ctx_poll_status", "dit_debug_tap", "dit_debug_poison", "dit_debug_check_guards", "dit_debug_expire_wait", "dit_debug_clock_probe", "dit_ctx_set_timing", "dit_ctx_read_timing", "dit_modulation_noalloc",
           "dit_load_shell_weights", "dit_timestep_cond", "dit_embed_latents", "dit_final_layer", "dit_sampler_update",
           "dit_denoise_step", "dit_denoise_round", "dit_last_launch_count", "dit_status_string", "dit_last_error"]


class DitConfig(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("mlp_hidden", C.c_int32),
                ("cond_dim", C.c_int32), ("max_blocks", C.c_int32), ("max_total_tokens", C.c_int32),
                ("max_requests", C.c_int32), ("ln_eps", C.c_float), ("flags", C.c_uint32)]


class DitRequest(C.Structure):
    _fields_ = [("height", C.c_int32), ("width", C.c_int32), ("n_text_tokens", C.c_int32),
                ("timestep", C.c_float), ("step_index", C.c_int32)]


class DitBlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_o", "b_o",
                                          "w_fc1", "b_fc1", "w_fc2", "b_fc2", "q_norm", "k_norm")]


class DitParallelBlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_fc1", "b_fc1", "w_out", "b_out",
                                          "q_norm", "k_norm")]


class DitShellWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_in", "b_in", "w_t1", "b_t1", "w_t2", "b_t2", "w_fa", "b_fa",
                                          "w_out", "b_out")]


SCHED_EXPORTS = ["dit_sched_allocate", "dit_sched_round"]


class DitSchedOption(C.Structure):
    _fields_ = [("steps", C.c_int32), ("gpus", C.c_int32), ("step_time", C.c_double)]


class DitSchedRequest(C.Structure):
    _fields_ = [("options", C.POINTER(DitSchedOption)), ("n_options", C.c_int32), ("t_min", C.c_double),
                ("deadline", C.c_double)]


class DitError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {detail}" if detail else name)


_lib = None


def load_library() -> C.CDLL:
    """Loads libdit.so and declares the signatures of include/dit.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_01565_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.dit_workspace_bytes.restype = C.c_size_t
    lib.dit_workspace_bytes.argtypes = [C.POINTER(DitConfig)]
    lib.dit_ctx_create.restype = C.c_int
    lib.dit_ctx_create.argtypes = [C.POINTER(DitConfig), vp, C.c_size_t, C.POINTER(vp)]
    lib.dit_ctx_destroy.restype = C.c_int
    lib.dit_ctx_destroy.argtypes = [vp]
    lib.dit_load_block_weights.restype = C.c_int
    lib.dit_load_block_weights.argtypes = [vp, i32, C.POINTER(DitBlockWeights), vp]
    lib.dit_load_dual_block_weights.restype = C.c_int
    lib.dit_load_dual_block_weights.argtypes = [vp, i32, C.POINTER(DitBlockWeights), C.POINTER(DitBlockWeights), vp]
    lib.dit_load_parallel_block_weights.restype = C.c_int
    lib.dit_load_parallel_block_weights.argtypes = [vp, i32, C.POINTER(DitParallelBlockWeights), vp]
    lib.dit_pack_requests.restype = C.c_int
    lib.dit_pack_requests.argtypes = [C.POINTER(DitRequest), i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32),
                                      C.POINTER(i32), C.POINTER(i32)]
    lib.dit_pack_tokens.restype = C.c_int
    lib.dit_pack_tokens.argtypes = [vp, C.POINTER(vp), C.POINTER(i32), i32, vp, vp]
    lib.dit_step_forward.restype = C.c_int
    lib.dit_step_forward.argtypes = [vp, vp, C.POINTER(i32), i32, vp, i32, vp, vp]
    lib.dit_step_forward_host.restype = C.c_int
    lib.dit_step_forward_host.argtypes = [vp, vp, C.POINTER(i32), i32, vp, i32, vp, vp]
    lib.dit_step_forward_host_async.restype = C.c_int
    lib.dit_step_forward_host_async.argtypes = [vp, vp, C.POINTER(i32), i32, vp, i32, vp, vp]
    lib.dit_host_wait.restype = C.c_int
    lib.dit_host_wait.argtypes = [vp, i32]
    lib.dit_ctx_poll_status.restype = C.c_int
    lib.dit_ctx_poll_status.argtypes = [vp]
    lib.dit_debug_tap.restype = C.c_int
    lib.dit_debug_tap.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(i64), C.POINTER(i64), C.POINTER(i32)]
    lib.dit_debug_poison.restype = C.c_int
    lib.dit_debug_poison.argtypes = [vp, vp]
    lib.dit_debug_check_guards.restype = C.c_int
    lib.dit_debug_check_guards.argtypes = [vp, C.POINTER(i32)]
    lib.dit_debug_expire_wait.restype = C.c_int
    lib.dit_debug_expire_wait.argtypes = [vp, vp]
    lib.dit_debug_clock_probe.restype = C.c_int
    lib.dit_debug_clock_probe.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.dit_ctx_set_timing.restype = C.c_int
    lib.dit_ctx_set_timing.argtypes = [vp, i32]
    lib.dit_ctx_read_timing.restype = C.c_int
    lib.dit_ctx_read_timing.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.dit_modulation_noalloc.restype = C.c_int
    lib.dit_modulation_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
    fp = C.POINTER(C.c_float)
    rq = C.POINTER(DitRequest)
    lib.dit_step_forward_requests.restype = C.c_int
    lib.dit_step_forward_requests.argtypes = [vp, vp, rq, i32, vp, i32, vp, vp]
    lib.dit_load_shell_weights.restype = C.c_int
    lib.dit_load_shell_weights.argtypes = [vp, C.POINTER(DitShellWeights), vp]
    lib.dit_timestep_cond.restype = C.c_int
    lib.dit_timestep_cond.argtypes = [vp, rq, i32, vp, vp, vp]
    lib.dit_embed_latents.restype = C.c_int
    lib.dit_embed_latents.argtypes = [vp, vp, vp, rq, i32, vp, vp]
    lib.dit_final_layer.restype = C.c_int
    lib.dit_final_layer.argtypes = [vp, vp, rq, i32, vp, vp, vp]
    lib.dit_sampler_update.restype = C.c_int
    lib.dit_sampler_update.argtypes = [vp, vp, vp, rq, i32, fp, vp]
    lib.dit_denoise_step.restype = C.c_int
    lib.dit_denoise_step.argtypes = [vp, vp, vp, rq, i32, fp, vp, i32, vp, vp]
    lib.dit_denoise_round.restype = C.c_int
    lib.dit_denoise_round.argtypes = [vp, vp, vp, rq, i32, C.POINTER(i32), fp, i32, vp, i32, vp]
    lib.dit_sched_allocate.restype = C.c_int
    lib.dit_sched_allocate.argtypes = [C.POINTER(i32), C.POINTER(C.c_double), i32, i32, C.c_double,
                                       C.POINTER(DitSchedOption), C.POINTER(i32), C.POINTER(C.c_double), C.POINTER(i32)]
    lib.dit_sched_round.restype = C.c_int
    lib.dit_sched_round.argtypes = [C.POINTER(DitSchedRequest), i32, i32, C.c_double, C.c_double, C.POINTER(i32),
                                    C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.dit_last_launch_count.restype = i64
    lib.dit_last_launch_count.argtypes = [vp]
    lib.dit_status_string.restype = C.c_char_p
    lib.dit_status_string.argtypes = [C.c_int]
    lib.dit_last_error.restype = C.c_char_p
    lib.dit_last_error.argtypes = [vp]
    _lib = lib
    return lib


def dit_sched_allocate(gpus: Sequence[int], step_time: Sequence[float], steps: int, time_budget: float):
    """Returns (options [(steps, gpus, step_time)], gpu_time, feasible)."""
    lib = load_library()
    n = len(gpus)
    g = (C.c_int32 * n)(*gpus)
    t = (C.c_double * n)(*step_time)
    out = (DitSchedOption * 2)()
    n_out, feasible, cost = C.c_int32(), C.c_int32(), C.c_double()
    st = lib.dit_sched_allocate(g, t, n, steps, time_budget, out, C.byref(n_out), C.byref(cost), C.byref(feasible))
    if st != DIT_OK:
        raise DitError(st)
    return [(out[i].steps, out[i].gpus, out[i].step_time) for i in range(n_out.value)], cost.value, bool(feasible.value)


def dit_sched_round(reqs, n_gpus: int, tau: float, t_now: float):
    """reqs: list of (options [(steps, gpus, step_time)], t_min, deadline).
    Returns (chosen option per request or -1, steps done per request, survivors, gpus used)."""
    lib = load_library()
    n = len(reqs)
    keep = []
    arr = (DitSchedRequest * max(n, 1))()
    for i, (options, t_min, deadline) in enumerate(reqs):
        o = (DitSchedOption * max(len(options), 1))(*[DitSchedOption(int(s), int(a), float(t)) for (s, a, t) in options])
        keep.append(o)
        arr[i] = DitSchedRequest(o, len(options), float(t_min), float(deadline))
    chosen = (C.c_int32 * max(n, 1))()
    done = (C.c_int32 * max(n, 1))()
    surv, used = C.c_int32(), C.c_int32()
    st = lib.dit_sched_round(arr, n, n_gpus, tau, t_now, chosen, done, C.byref(surv), C.byref(used))
    if st != DIT_OK:
        raise DitError(st)
    return list(chosen[:n]), list(done[:n]), surv.value, used.value


def request_array(reqs: Sequence) -> "C.Array":
    """reqs: (height, width, n_text[, timestep, step_index]) tuples, or objects with those attributes."""
    arr = (DitRequest * max(len(reqs), 1))()
    for i, r in enumerate(reqs):
        if hasattr(r, "height"):
            arr[i] = DitRequest(int(r.height), int(r.width), int(r.n_text_tokens), float(r.timestep), int(r.step_index))
        else:
            arr[i] = DitRequest(int(r[0]), int(r[1]), int(r[2]), float(r[3]) if len(r) > 3 else 0.0,
                                int(r[4]) if len(r) > 4 else 0)
    return arr


def dit_pack_requests(reqs: Sequence[Sequence]) -> Dict[str, np.ndarray]:
    """reqs: (height, width, n_text[, timestep, step_index]).  Host-only; returns int32 arrays."""
    lib = load_library()
    n = len(reqs)
    arr = (DitRequest * max(n, 1))()
    for i, r in enumerate(reqs):
        arr[i] = DitRequest(int(r[0]), int(r[1]), int(r[2]), float(r[3]) if len(r) > 3 else 0.0,
                            int(r[4]) if len(r) > 4 else 0)
    lens = np.zeros(max(n, 1), dtype=np.int32)
    cu = np.zeros(n + 1, dtype=np.int32)
    total = C.c_int32(0)
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    st = lib.dit_pack_requests(arr, n, ip(lens), ip(cu), None, None, C.byref(total))
    if st != DIT_OK:
        raise DitError(st)
    row_req = np.zeros(max(total.value, 1), dtype=np.int32)
    row_local = np.zeros(max(total.value, 1), dtype=np.int32)
    st = lib.dit_pack_requests(arr, n, ip(lens), ip(cu), ip(row_req), ip(row_local), C.byref(total))
    if st != DIT_OK:
        raise DitError(st)
    return {"token_lens": lens[:n], "cu_seqlens": cu, "row_req": row_req[:total.value],
            "row_local": row_local[:total.value], "total_tokens": total.value}


class DitContext:
    """Owns a workspace tensor and a dit_ctx on the current CUDA device."""

    def __init__(self, hidden: int, n_heads: int, head_dim: int, mlp_hidden: int, cond_dim: int,
                 max_blocks: int, max_total_tokens: int, max_requests: int = 8, ln_eps: float = 1e-6,
                 flags: int = 0):
        import torch
        self.torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("libdit needs a CUDA device (sm_100); there is no CPU path")
        self.cfg = DitConfig(hidden, n_heads, head_dim, mlp_hidden, cond_dim, max_blocks, max_total_tokens,
                             max_requests, ln_eps, flags)
        nbytes = self.lib.dit_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise DitError(2, "configuration rejected by dit_workspace_bytes")
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.workspace_bytes = nbytes
        handle = C.c_void_p()
        st = self.lib.dit_ctx_create(C.byref(self.cfg), C.c_void_p(base), nbytes, C.byref(handle))
        if st != DIT_OK:
            raise DitError(st, "dit_ctx_create")
        self.handle = handle
        self.hidden, self.cond_dim, self.mlp_hidden = hidden, cond_dim, mlp_hidden

    # ------------------------------------------------------------------ helpers
    def _check(self, st: int):
        if st != DIT_OK:
            raise DitError(st, self.lib.dit_last_error(self.handle).decode())

    def _stream(self, stream=None) -> C.c_void_p:
        s = self.torch.cuda.current_stream() if stream is None else stream
        return C.c_void_p(s.cuda_stream)

    @staticmethod
    def _lens(lens) -> np.ndarray:
        return np.ascontiguousarray(np.asarray(lens, dtype=np.int32))

    def close(self):
        if getattr(self, "handle", None) is not None:
            self.torch.cuda.synchronize()
            self.lib.dit_ctx_destroy(self.handle)
            self.handle = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ C-ABI calls
    def _block_struct(self, weights: Dict[str, "object"]) -> DitBlockWeights:
        w = DitBlockWeights()
        for name, _ in DitBlockWeights._fields_:
            t = weights.get(name)
            if t is None:
                setattr(w, name, None)
                continue
            assert t.is_cuda and t.dtype == self.torch.bfloat16 and t.is_contiguous(), name
            setattr(w, name, t.data_ptr())
        return w

    def dit_load_block_weights(self, block_idx: int, weights: Dict[str, "object"], stream=None):
        """weights: name -> CUDA bf16 tensor, [in, out] row-major; biases may be None."""
        w = self._block_struct(weights)
        self._check(self.lib.dit_load_block_weights(self.handle, block_idx, C.byref(w), self._stream(stream)))

    def dit_load_dual_block_weights(self, block_idx: int, image_stream: Dict[str, "object"],
                                    text_stream: Dict[str, "object"], stream=None):
        """Two-stream block in slots block_idx (image tokens) and block_idx + 1 (text tokens)."""
        wi, wt = self._block_struct(image_stream), self._block_struct(text_stream)
        self._check(self.lib.dit_load_dual_block_weights(self.handle, block_idx, C.byref(wi), C.byref(wt), self._stream(stream)))

    def dit_load_parallel_block_weights(self, block_idx: int, weights: Dict[str, "object"], stream=None):
        """Parallel-form block: name -> CUDA bf16 tensor ([in, out] row-major); biases and norms may be None."""
        w = DitParallelBlockWeights()
        keep = []
        for name, _ in DitParallelBlockWeights._fields_:
            t = weights.get(name)
            if t is not None:
                assert t.is_cuda and t.dtype == self.torch.bfloat16 and t.is_contiguous(), name
                keep.append(t)
            setattr(w, name, t.data_ptr() if t is not None else None)
        self._check(self.lib.dit_load_parallel_block_weights(self.handle, block_idx, C.byref(w), self._stream(stream)))

    def dit_pack_tokens(self, per_request_tokens: List["object"], stream=None):
        torch = self.torch
        n = len(per_request_tokens)
        lens = self._lens([t.shape[0] for t in per_request_tokens])
        for t in per_request_tokens:
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape[1] == self.hidden
        packed = torch.empty((int(lens.sum()), self.hidden), dtype=torch.bfloat16, device="cuda")
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in per_request_tokens])
        self._check(self.lib.dit_pack_tokens(self.handle, ptrs, lens.ctypes.data_as(C.POINTER(C.c_int32)), n,
                                             C.c_void_p(packed.data_ptr()), self._stream(stream)))
        return packed

    def dit_step_forward(self, packed_tokens, token_lens, cond, n_blocks: int, out=None, stream=None):
        """packed_tokens [T,H] bf16 cuda, cond [R,C] bf16 cuda -> out [T,H] fp32 cuda (asynchronous)."""
        torch = self.torch
        lens = self._lens(token_lens)
        assert packed_tokens.is_cuda and packed_tokens.dtype == torch.bfloat16 and packed_tokens.is_contiguous()
        assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous()
        assert packed_tokens.shape == (int(lens.sum()), self.hidden) and cond.shape == (len(lens), self.cond_dim)
        if out is None:
            out = torch.empty(packed_tokens.shape, dtype=torch.float32, device="cuda")
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.shape == packed_tokens.shape
        self._check(self.lib.dit_step_forward(self.handle, C.c_void_p(packed_tokens.data_ptr()),
                                              lens.ctypes.data_as(C.POINTER(C.c_int32)), len(lens),
                                              C.c_void_p(cond.data_ptr()), n_blocks, C.c_void_p(out.data_ptr()),
                                              self._stream(stream)))
        return out

    def dit_step_forward_requests(self, packed_tokens, reqs, cond, n_blocks: int, out=None, stream=None):
        """dit_step_forward with the batch given as requests (needed by the rotary term)."""
        torch = self.torch
        assert packed_tokens.is_cuda and packed_tokens.dtype == torch.bfloat16 and packed_tokens.is_contiguous()
        assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous()
        assert packed_tokens.shape[1] == self.hidden and cond.shape == (len(reqs), self.cond_dim)
        if out is None:
            out = torch.empty(packed_tokens.shape, dtype=torch.float32, device="cuda")
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.shape == packed_tokens.shape
        self._check(self.lib.dit_step_forward_requests(self.handle, self._ptr(packed_tokens), request_array(reqs), len(reqs),
                                                       self._ptr(cond), n_blocks, self._ptr(out), self._stream(stream)))
        return out

    def dit_step_forward_host(self, host_tokens, token_lens, host_cond, n_blocks: int, host_out, stream=None):
        """Host (ideally pinned) torch tensors in and out; returns after `out` is valid."""
        lens = self._lens(token_lens)
        assert not host_tokens.is_cuda and not host_cond.is_cuda and not host_out.is_cuda
        assert host_tokens.is_contiguous() and host_cond.is_contiguous() and host_out.is_contiguous()
        assert host_tokens.shape == (int(lens.sum()), self.hidden) and host_out.shape == host_tokens.shape
        self._check(self.lib.dit_step_forward_host(self.handle, C.c_void_p(host_tokens.data_ptr()),
                                                   lens.ctypes.data_as(C.POINTER(C.c_int32)), len(lens),
                                                   C.c_void_p(host_cond.data_ptr()), n_blocks,
                                                   C.c_void_p(host_out.data_ptr()), self._stream(stream)))
        return host_out

    def dit_step_forward_host_async(self, host_tokens, token_lens, host_cond, n_blocks: int, host_out, stream=None):
        """The same without the final wait; dit_host_wait(0 or 1) covers the latest call or the one before."""
        lens = self._lens(token_lens)
        assert not host_tokens.is_cuda and not host_cond.is_cuda and not host_out.is_cuda
        assert host_tokens.is_contiguous() and host_cond.is_contiguous() and host_out.is_contiguous()
        assert host_tokens.shape == (int(lens.sum()), self.hidden) and host_out.shape == host_tokens.shape
        self._check(self.lib.dit_step_forward_host_async(self.handle, C.c_void_p(host_tokens.data_ptr()),
                                                         lens.ctypes.data_as(C.POINTER(C.c_int32)), len(lens),
                                                         C.c_void_p(host_cond.data_ptr()), n_blocks,
                                                         C.c_void_p(host_out.data_ptr()), self._stream(stream)))
        return host_out

    def dit_host_wait(self, calls_back: int = 0):
        self._check(self.lib.dit_host_wait(self.handle, calls_back))

    # ------------------------------------------------------------------ shell around the block stack
    @staticmethod
    def _ptr(t) -> C.c_void_p:
        return C.c_void_p(t.data_ptr()) if t is not None else None

    def _f32(self, t, n=None):
        assert t.is_cuda and t.dtype == self.torch.float32 and t.is_contiguous()
        assert n is None or t.numel() == n
        return t

    def dit_load_shell_weights(self, weights: Dict[str, "object"], stream=None):
        """weights: name -> CUDA bf16 tensor, [in, out] row-major; biases may be None."""
        w = DitShellWeights()
        keep = []
        for name, _ in DitShellWeights._fields_:
            t = weights.get(name)
            if t is not None:
                assert t.is_cuda and t.dtype == self.torch.bfloat16 and t.is_contiguous(), name
                keep.append(t)
            setattr(w, name, t.data_ptr() if t is not None else None)
        self._check(self.lib.dit_load_shell_weights(self.handle, C.byref(w), self._stream(stream)))

    def dit_timestep_cond(self, reqs, pooled=None, cond_out=None, stream=None):
        """-> cond [n, C] bf16 cuda.  pooled: [n, C] fp32 cuda or None."""
        torch = self.torch
        n = len(reqs)
        if pooled is not None:
            self._f32(pooled, n * self.cond_dim)
        if cond_out is None:
            cond_out = torch.empty((n, self.cond_dim), dtype=torch.bfloat16, device="cuda")
        self._check(self.lib.dit_timestep_cond(self.handle, request_array(reqs), n, self._ptr(pooled),
                                               self._ptr(cond_out), self._stream(stream)))
        return cond_out

    def dit_embed_latents(self, latents, text_tokens, reqs, packed_tokens=None, stream=None):
        """latents: flat fp32 cuda (requests concatenated); text_tokens: [sum n_text, H] bf16 cuda or None."""
        torch = self.torch
        n = len(reqs)
        arr = request_array(reqs)
        n_img = sum((arr[i].height // 16) * (arr[i].width // 16) for i in range(n))
        n_txt = sum(arr[i].n_text_tokens for i in range(n))
        self._f32(latents, 64 * n_img)
        if text_tokens is not None:
            assert text_tokens.is_cuda and text_tokens.dtype == torch.bfloat16 and text_tokens.is_contiguous()
            assert text_tokens.shape == (n_txt, self.hidden)
        if packed_tokens is None:
            packed_tokens = torch.empty((n_img + n_txt, self.hidden), dtype=torch.bfloat16, device="cuda")
        self._check(self.lib.dit_embed_latents(self.handle, self._ptr(latents), self._ptr(text_tokens), arr, n,
                                               self._ptr(packed_tokens), self._stream(stream)))
        return packed_tokens

    def dit_final_layer(self, x, reqs, cond, velocity=None, stream=None):
        """x [T, H] fp32 cuda, cond [n, C] bf16 cuda -> velocity, flat fp32 cuda in latent layout."""
        torch = self.torch
        n = len(reqs)
        arr = request_array(reqs)
        n_img = sum((arr[i].height // 16) * (arr[i].width // 16) for i in range(n))
        self._f32(x)
        assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous() and cond.shape == (n, self.cond_dim)
        if velocity is None:
            velocity = torch.empty(64 * n_img, dtype=torch.float32, device="cuda")
        self._f32(velocity, 64 * n_img)
        self._check(self.lib.dit_final_layer(self.handle, self._ptr(x), arr, n, self._ptr(cond), self._ptr(velocity),
                                             self._stream(stream)))
        return velocity

    def dit_sampler_update(self, latents, velocity, reqs, dsigma, stream=None):
        n = len(reqs)
        ds = np.ascontiguousarray(np.asarray(dsigma, dtype=np.float32))
        assert ds.shape == (n,)
        self._f32(latents)
        self._f32(velocity, latents.numel())
        self._check(self.lib.dit_sampler_update(self.handle, self._ptr(latents), self._ptr(velocity), request_array(reqs), n,
                                                ds.ctypes.data_as(C.POINTER(C.c_float)), self._stream(stream)))
        return latents

    def dit_denoise_step(self, latents, text_tokens, reqs, dsigma, pooled, n_blocks: int, velocity=None, stream=None):
        """One full step in place on `latents` (flat fp32 cuda).  Returns latents."""
        n = len(reqs)
        ds = np.ascontiguousarray(np.asarray(dsigma, dtype=np.float32))
        assert ds.shape == (n,)
        self._f32(latents)
        if velocity is not None:
            self._f32(velocity, latents.numel())
        if pooled is not None:
            self._f32(pooled, n * self.cond_dim)
        self._check(self.lib.dit_denoise_step(self.handle, self._ptr(latents), self._ptr(text_tokens), request_array(reqs), n,
                                              ds.ctypes.data_as(C.POINTER(C.c_float)), self._ptr(pooled), n_blocks,
                                              self._ptr(velocity), self._stream(stream)))
        return latents

    def dit_denoise_round(self, latents, text_tokens, reqs, steps_in_round, sigmas, pooled, n_blocks: int, stream=None):
        """steps_in_round: [n] ints; sigmas: [n, max_steps + 1] floats (host).  Latents updated in place."""
        n = len(reqs)
        steps = np.ascontiguousarray(np.asarray(steps_in_round, dtype=np.int32))
        sig = np.ascontiguousarray(np.asarray(sigmas, dtype=np.float32))
        assert steps.shape == (n,) and sig.ndim == 2 and sig.shape[0] == n
        self._f32(latents)
        if pooled is not None:
            self._f32(pooled, n * self.cond_dim)
        self._check(self.lib.dit_denoise_round(self.handle, self._ptr(latents), self._ptr(text_tokens), request_array(reqs), n,
                                               steps.ctypes.data_as(C.POINTER(C.c_int32)),
                                               sig.ctypes.data_as(C.POINTER(C.c_float)), sig.shape[1], self._ptr(pooled),
                                               n_blocks, self._stream(stream)))
        return latents

    def dit_ctx_poll_status(self):
        self._check(self.lib.dit_ctx_poll_status(self.handle))

    def dit_debug_poison(self, stream=None):
        """Fills the activation regions of the workspace with NaN bytes and rewrites the guard areas."""
        self._check(self.lib.dit_debug_poison(self.handle, self._stream(stream)))

    def dit_debug_check_guards(self) -> int:
        """Number of damaged guard areas (0 after a correct step)."""
        n = C.c_int32(-1)
        self._check(self.lib.dit_debug_check_guards(self.handle, C.byref(n)))
        return int(n.value)

    def dit_debug_expire_wait(self, stream=None):
        """Launches the one-CTA kernel whose bounded wait runs out (sets the status word)."""
        self._check(self.lib.dit_debug_expire_wait(self.handle, self._stream(stream)))

    def dit_debug_clock_probe(self, enabled: bool):
        """Sets the probe's state; returns (SM MHz inside an attention CTA, its cycles per key block, SM MHz inside a
        GEMM CTA) left since the last call."""
        mhz, cyc, gmhz = C.c_int32(0), C.c_int32(0), C.c_int32(0)
        self._check(self.lib.dit_debug_clock_probe(self.handle, 1 if enabled else 0, C.byref(mhz), C.byref(cyc), C.byref(gmhz)))
        return int(mhz.value), int(cyc.value), int(gmhz.value)

    def dit_ctx_set_timing(self, enabled: bool):
        self._check(self.lib.dit_ctx_set_timing(self.handle, 1 if enabled else 0))

    def dit_ctx_read_timing(self) -> Dict[str, Dict[str, float]]:
        ms = (C.c_double * len(KERNEL_KINDS))()
        n = (C.c_int64 * len(KERNEL_KINDS))()
        self._check(self.lib.dit_ctx_read_timing(self.handle, ms, n))
        return {k: {"ms": ms[i], "launches": int(n[i])} for i, k in enumerate(KERNEL_KINDS)}

    def dit_last_launch_count(self) -> int:
        return int(self.lib.dit_last_launch_count(self.handle))

    def dit_debug_tap(self, which: str):
        """Copy of an internal buffer of the last step as a torch tensor (fp16, bf16 in the bf16-operand mode, or fp32)."""
        torch = self.torch
        ptr, rows, cols, eb = C.c_void_p(), C.c_int64(), C.c_int64(), C.c_int32()
        self._check(self.lib.dit_debug_tap(self.handle, TAPS[which], C.byref(ptr), C.byref(rows), C.byref(cols), C.byref(eb)))
        dtype16 = torch.bfloat16 if (self.cfg.flags & DIT_FLAG_BF16_OPERANDS) else torch.float16
        dtype = dtype16 if eb.value == 2 else torch.float32
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        off = ptr.value - base
        torch.cuda.synchronize()
        flat = self.workspace[(base - self.workspace.data_ptr()) + off:(base - self.workspace.data_ptr()) + off + rows.value * cols.value * eb.value]
        return flat.view(dtype).view(rows.value, cols.value).clone()


def dit_modulation_noalloc(cond, w_ada, b_ada, mod_out, stream=None):
    """cond [R,C], w_ada [C,6H], b_ada [6H] or None: CUDA bf16 tensors; mod_out [R,6H] CUDA fp32, written in place.

    Marshalling only: the caller provides every buffer, nothing is allocated here or in the library.
    """
    import torch
    lib = load_library()
    R, Cd = cond.shape
    H = w_ada.shape[1] // 6
    assert cond.is_cuda and cond.dtype == torch.bfloat16 and cond.is_contiguous()
    assert w_ada.is_cuda and w_ada.dtype == torch.bfloat16 and w_ada.is_contiguous() and w_ada.shape == (Cd, 6 * H)
    assert b_ada is None or (b_ada.is_cuda and b_ada.dtype == torch.bfloat16 and b_ada.shape == (6 * H,))
    assert mod_out.is_cuda and mod_out.dtype == torch.float32 and mod_out.is_contiguous() and mod_out.shape == (R, 6 * H)
    s = torch.cuda.current_stream() if stream is None else stream
    st = lib.dit_modulation_noalloc(C.c_void_p(cond.data_ptr()), C.c_void_p(w_ada.data_ptr()),
                                    C.c_void_p(b_ada.data_ptr()) if b_ada is not None else None, R, Cd, H,
                                    C.c_void_p(mod_out.data_ptr()), C.c_void_p(s.cuda_stream))
    if st != DIT_OK:
        raise DitError(st, lib.dit_status_string(st).decode())
    return mod_out


def context_for(dims, max_blocks: int, max_total_tokens: int, max_requests: int = 8, flags: int = 0) -> DitContext:
    return DitContext(dims.hidden, dims.n_heads, dims.head_dim, dims.mlp_hidden, dims.cond_dim,
                      max_blocks, max_total_tokens, max_requests, dims.ln_eps, flags)


def upload_weights(ctx: DitContext, blocks) -> int:
    """blocks: list of dicts name -> numpy uint16 (bf16 bits).  Copies to the GPU and loads them.

    A dict with "w_out" is a parallel-form block; a dict with "txt" (the text stream's dict) is a
    two-stream block and takes two slots.  Returns the number of slots used (n_blocks of a step).
    """
    import torch
    to_dev = lambda w: {k: torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16) for k, v in w.items() if k != "txt"}
    slot = 0
    for w in blocks:
        dev = to_dev(w)
        if "txt" in w:
            txt = to_dev(w["txt"])
            ctx.dit_load_dual_block_weights(slot, dev, txt)
            slot += 2
        elif "w_out" in w:
            ctx.dit_load_parallel_block_weights(slot, dev)
            slot += 1
        else:
            ctx.dit_load_block_weights(slot, dev)
            slot += 1
        torch.cuda.synchronize()
        del dev
    return slot


def upload_shell_weights(ctx: DitContext, shell) -> None:
    """shell: dict name -> numpy uint16 (bf16 bits)."""
    import torch
    dev = {k: torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16) for k, v in shell.items()}
    ctx.dit_load_shell_weights(dev)
    torch.cuda.synchronize()


def bits_to_cuda_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
