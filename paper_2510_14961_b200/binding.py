"""ctypes binding of the C ABI in include/rd.h.  Argument marshalling only: every step of the path
runs inside the CUDA library.  There is no CPU fallback: a missing or unloadable library raises."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librd_b200.so")

RD_F32, RD_BF16 = 0, 1
RD_OK, RD_E_INVALID_ARG, RD_E_STATE, RD_E_CAPACITY, RD_E_OOM, RD_E_CUDA, RD_E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
RD_DBG_LATENTS, RD_DBG_DELTA, RD_DBG_DRAFTS, RD_DBG_LOGITS, RD_DBG_EMBED = 0, 1, 2, 3, 4

EXPORTS = ["rd_load", "rd_free", "rd_session_create", "rd_session_destroy", "rd_prefill", "rd_ar_step",
           "rd_df_step", "rd_sync", "rd_committed", "rd_get_tokens", "rd_last_step_rows", "rd_debug_read",
           "rd_debug_force_tokens", "rd_debug_read_kv", "rd_stats", "rd_set_gemm_path", "rd_strerror",
           "rd_last_cuda_error", "rd_profile_enable", "rd_profile_read", "rd_debug_read_kv_noalloc", "rd_set_launch_chaining",
           "rd_debug_expire_next_wait", "rd_set_fused_swiglu", "rd_set_attention_path", "rd_poll_begin", "rd_poll_end",
           "rd_debug_gemm_sequence", "rd_prefill_sliced", "rd_prefill_advance", "rd_prefill_pending",
           "rd_set_prefill_units"]


class RdConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("hidden", "n_heads", "head_dim", "mlp_inner", "n_prelude", "n_core",
                                         "n_coda", "vocab", "dtype", "tie_embeddings")] + \
               [(n, C.c_float) for n in ("rope_base", "norm_eps", "init_sigma")]


class RdSessionConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "max_context", "max_window", "max_iters_per_pos",
                                         "max_new_tokens", "keep_logits")] + \
               [("temperature", C.c_float), ("seed", C.c_uint64), ("eta", C.c_float), ("beta", C.c_float),
                ("top_p", C.c_float), ("latent_slots", C.c_int32)]


class RdStats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("df_steps", "ar_steps", "rows_prelude", "rows_core", "rows_coda",
                                          "tokens_committed", "kernel_launches", "tc_gemm_launches",
                                          "weight_bytes", "kv_bytes", "flops")] + [("commit_hist", C.c_uint64 * 16)]


class RdProfile(C.Structure):
    _fields_ = [("gemm_launches", C.c_uint64), ("gemm_ms", C.c_double), ("gemm_weight_bytes", C.c_uint64),
                ("attn_launches", C.c_uint64), ("attn_ms", C.c_double), ("attn_kv_bytes", C.c_uint64),
                ("other_launches", C.c_uint64), ("other_ms", C.c_double)]


class RdError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {code} ({detail})")


_lib = None


def lib():
    """The loaded library (raises if it is missing: build it with paper_2510_14961_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2510_14961_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        L.rd_load.argtypes = [C.POINTER(RdConfig), C.POINTER(vp), i32, i32, C.POINTER(vp)]
        L.rd_free.argtypes = [vp]
        L.rd_free.restype = None
        L.rd_session_create.argtypes = [vp, C.POINTER(RdSessionConfig), vp, C.POINTER(vp)]
        L.rd_session_destroy.argtypes = [vp]
        L.rd_session_destroy.restype = None
        L.rd_prefill.argtypes = [vp, i32, vp, i32, i32]
        L.rd_prefill_sliced.argtypes = [vp, i32, vp, i32, i32]
        L.rd_prefill_advance.argtypes = [vp, i32]
        L.rd_prefill_pending.argtypes = [vp]
        L.rd_set_prefill_units.argtypes = [vp, i32]
        L.rd_ar_step.argtypes = [vp, i32]
        L.rd_df_step.argtypes = [vp, i32, i32, f32]
        L.rd_sync.argtypes = [vp]
        L.rd_committed.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32)]
        L.rd_get_tokens.argtypes = [vp, i32, vp, i32, C.POINTER(i32)]
        L.rd_last_step_rows.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32)]
        L.rd_debug_read.argtypes = [vp, i32, i32, vp, C.c_size_t]
        L.rd_debug_force_tokens.argtypes = [vp, i32, i32, vp, i32]
        L.rd_debug_read_kv.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp]
        L.rd_debug_read_kv_noalloc.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp]
        L.rd_stats.argtypes = [vp, C.POINTER(RdStats)]
        L.rd_set_gemm_path.argtypes = [vp, i32]
        L.rd_set_launch_chaining.argtypes = [vp, i32]
        L.rd_debug_expire_next_wait.argtypes = [vp]
        L.rd_set_fused_swiglu.argtypes = [vp, i32]
        L.rd_set_attention_path.argtypes = [vp, i32]
        L.rd_debug_gemm_sequence.argtypes = [vp, i32, i32, C.POINTER(C.c_uint64), C.POINTER(i32)]
        L.rd_poll_begin.argtypes = [vp, C.POINTER(i32)]
        L.rd_poll_end.argtypes = [vp, i32, i32, C.POINTER(i32), C.POINTER(i32)]
        L.rd_profile_enable.argtypes = [vp, i32]
        L.rd_profile_read.argtypes = [vp, C.POINTER(RdProfile)]
        L.rd_strerror.argtypes = [C.c_int]
        L.rd_strerror.restype = C.c_char_p
        L.rd_last_cuda_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(rc, where):
    if rc != RD_OK:
        L = lib()
        detail = L.rd_strerror(rc).decode()
        if rc in (RD_E_CUDA, RD_E_OOM):
            detail += "; " + L.rd_last_cuda_error().decode()
        raise RdError(rc, where, detail)


def _ptr(x):
    """Address of a numpy array (host) or of anything exposing data_ptr() (a torch tensor)."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data


class Model:
    """rd_load: device copy of the weights of P, R and C."""

    def __init__(self, hidden, n_heads, head_dim, mlp_inner, n_prelude, n_core, n_coda, vocab, tensors,
                 dtype=RD_F32, tie_embeddings=True, rope_base=10000.0, norm_eps=1e-6, init_sigma=1.0,
                 elem_bytes=4):
        """`tensors`: sequence of arrays in the order include/rd.h states (numpy on the host or torch
        tensors on the device); gains float32, matrices float32 (elem_bytes 4) or bf16 bits (2)."""
        self.cfg = RdConfig(hidden, n_heads, head_dim, mlp_inner, n_prelude, n_core, n_coda, vocab, dtype,
                            1 if tie_embeddings else 0, rope_base, norm_eps, init_sigma)
        self._keep = list(tensors)
        arr = (C.c_void_p * len(self._keep))(*[_ptr(t) for t in self._keep])
        self.handle = C.c_void_p()
        _check(lib().rd_load(C.byref(self.cfg), arr, len(self._keep), elem_bytes, C.byref(self.handle)), "rd_load")
        self._keep = None

    def close(self):
        if self.handle:
            lib().rd_free(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Session:
    """rd_session_create and the per-session calls."""

    def __init__(self, model: Model, batch=1, max_context=1024, max_window=1, max_iters_per_pos=64,
                 max_new_tokens=64, keep_logits=False, temperature=0.0, seed=0, stream=None, eta=0.0, beta=0.0,
                 top_p=0.0, latent_slots=0):
        self.model = model
        self.sc = RdSessionConfig(batch, max_context, max_window, max_iters_per_pos, max_new_tokens,
                                  1 if keep_logits else 0, temperature, seed, eta, beta, top_p, latent_slots)
        self.handle = C.c_void_p()
        _check(lib().rd_session_create(model.handle, C.byref(self.sc), C.c_void_p(stream or 0),
                                       C.byref(self.handle)), "rd_session_create")

    def close(self):
        if self.handle:
            lib().rd_session_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, seq, prompt, r):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        _check(lib().rd_prefill(self.handle, seq, p.ctypes.data, len(p), r), "rd_prefill")

    def prefill_sliced(self, seq, prompt, r):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        _check(lib().rd_prefill_sliced(self.handle, seq, p.ctypes.data, len(p), r), "rd_prefill_sliced")

    def prefill_advance(self, units):
        _check(lib().rd_prefill_advance(self.handle, units), "rd_prefill_advance")

    def prefill_pending(self):
        n = lib().rd_prefill_pending(self.handle)
        if n < 0:
            _check(n, "rd_prefill_pending")
        return n

    def set_prefill_units(self, units_per_step):
        _check(lib().rd_set_prefill_units(self.handle, units_per_step), "rd_set_prefill_units")

    def ar_step(self, r):
        _check(lib().rd_ar_step(self.handle, r), "rd_ar_step")

    def df_step(self, window, inner_iters, exit_threshold=0.0):
        _check(lib().rd_df_step(self.handle, window, inner_iters, exit_threshold), "rd_df_step")

    def sync(self):
        _check(lib().rd_sync(self.handle), "rd_sync")

    def committed(self, seq=0):
        n, d = C.c_int32(), C.c_int32()
        _check(lib().rd_committed(self.handle, seq, C.byref(n), C.byref(d)), "rd_committed")
        return n.value, bool(d.value)

    def poll_begin(self):
        t = C.c_int32()
        _check(lib().rd_poll_begin(self.handle, C.byref(t)), "rd_poll_begin")
        return t.value

    def poll_end(self, ticket, seq=-1):
        n, d = C.c_int32(), C.c_int32()
        _check(lib().rd_poll_end(self.handle, ticket, seq, C.byref(n), C.byref(d)), "rd_poll_end")
        return n.value, bool(d.value)

    def tokens(self, seq=0, out=None):
        cap = self.sc.max_context + 1
        buf = out if out is not None else np.empty(cap, dtype=np.int32)
        n = C.c_int32()
        _check(lib().rd_get_tokens(self.handle, seq, _ptr(buf), len(buf), C.byref(n)), "rd_get_tokens")
        return buf[: n.value]

    def last_step_rows(self, seq=0):
        f, n = C.c_int32(), C.c_int32()
        _check(lib().rd_last_step_rows(self.handle, seq, C.byref(f), C.byref(n)), "rd_last_step_rows")
        return f.value, n.value

    def debug_read(self, what, seq=0):
        _, n = self.last_step_rows(seq)
        c = self.model.cfg
        shape, dt = {RD_DBG_LATENTS: ((n, c.hidden), np.float32), RD_DBG_EMBED: ((n, c.hidden), np.float32),
                     RD_DBG_DELTA: ((n,), np.float32), RD_DBG_DRAFTS: ((n,), np.int32),
                     RD_DBG_LOGITS: ((n, c.vocab), np.float32)}[what]
        out = np.empty(shape, dtype=dt)
        _check(lib().rd_debug_read(self.handle, what, seq, out.ctypes.data, out.nbytes), "rd_debug_read")
        return out

    def force_tokens(self, seq, first_pos, tokens):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        _check(lib().rd_debug_force_tokens(self.handle, seq, first_pos, t.ctypes.data, len(t)),
               "rd_debug_force_tokens")

    def read_kv(self, block, layer, which, seq, pos0, n):
        out = np.empty((n, self.model.cfg.hidden), dtype=np.float32)
        _check(lib().rd_debug_read_kv(self.handle, block, layer, which, seq, pos0, n, out.ctypes.data),
               "rd_debug_read_kv")
        return out

    def read_kv_noalloc(self, block, layer, which, seq, pos0, n):
        """read_kv through the library's fixed staging array: no device allocation is made.  For
        callers that cannot allocate (device memory fully committed, or other streams must not be
        stalled); at most 1,048,576 values per call, calls on one device must not overlap."""
        out = np.empty((n, self.model.cfg.hidden), dtype=np.float32)
        _check(lib().rd_debug_read_kv_noalloc(self.handle, block, layer, which, seq, pos0, n, out.ctypes.data),
               "rd_debug_read_kv_noalloc")
        return out

    def stats(self):
        st = RdStats()
        _check(lib().rd_stats(self.handle, C.byref(st)), "rd_stats")
        out = {k: getattr(st, k) for k, _ in RdStats._fields_}
        out["commit_hist"] = [int(v) for v in st.commit_hist]
        return out

    def set_gemm_path(self, path):
        _check(lib().rd_set_gemm_path(self.handle, path), "rd_set_gemm_path")

    def set_launch_chaining(self, on):
        _check(lib().rd_set_launch_chaining(self.handle, 1 if on else 0), "rd_set_launch_chaining")

    def set_attention_path(self, path):
        _check(lib().rd_set_attention_path(self.handle, path), "rd_set_attention_path")

    def set_fused_swiglu(self, on):
        _check(lib().rd_set_fused_swiglu(self.handle, 1 if on else 0), "rd_set_fused_swiglu")

    def gemm_sequence(self, n_rows, reps=1):
        """Measurement aid: the GEMM launches of a decode step, back to back; returns (weight bytes, launches)."""
        b, n = C.c_uint64(), C.c_int32()
        _check(lib().rd_debug_gemm_sequence(self.handle, n_rows, reps, C.byref(b), C.byref(n)), "rd_debug_gemm_sequence")
        return b.value, n.value

    def expire_next_wait(self):
        """Test aid: the next tensor-core GEMM launch lets one bounded wait run out (RD_E_TIMEOUT at the next sync)."""
        _check(lib().rd_debug_expire_next_wait(self.handle), "rd_debug_expire_next_wait")

    def profile_enable(self, on=True):
        _check(lib().rd_profile_enable(self.handle, 1 if on else 0), "rd_profile_enable")

    def profile_read(self):
        pr = RdProfile()
        _check(lib().rd_profile_read(self.handle, C.byref(pr)), "rd_profile_read")
        return {k: getattr(pr, k) for k, _ in RdProfile._fields_}
