"""ctypes binding over the C-ABI library (``include/jd.h``): argument marshalling only.

Every step of the verification runs inside the library's CUDA kernels; torch is used
here for device buffers and streams and for nothing else.  If the shared library is
missing the binding raises: there is no CPU or eager fallback.

The module-level functions carry the C names (``jd_create``, ``jd_set_head``,
``jd_verify`` ...) and take raw pointers; :class:`Verifier` wraps them for callers that
hold torch tensors.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

# JD_LIBRARY selects another build of the same library (the phase-stamp build of build.py --stamps)
_LIB_PATH = os.environ.get("JD_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libjd_b200.so")
_lib = None

JD_OK, JD_ERR_INVALID_ARG, JD_ERR_UNSUPPORTED, JD_ERR_ARCH = 0, 1, 2, 3
JD_ERR_ALLOC, JD_ERR_CUDA, JD_ERR_TIMEOUT, JD_ERR_BAD_TOKEN = 4, 5, 6, 7
JD_DTYPE_F32, JD_DTYPE_BF16, JD_DTYPE_FP8_E4M3 = 0, 1, 2
JD_MODE_STANDARD, JD_MODE_JUDGE, JD_MODE_JUDGE_OR_STANDARD = 0, 1, 2
JD_RESAMPLE_RESIDUAL, JD_RESAMPLE_TARGET_P = 0, 1
JD_VARIANT_AUTO, JD_VARIANT_SIMT, JD_VARIANT_FUSED, JD_VARIANT_BATCHED = 0, 1, 2, 3
JD_RULE_SAMPLING, JD_RULE_TOPK = 0, 1
JD_NORM_NONE, JD_NORM_RMS = 0, 1

MODES = {"standard": JD_MODE_STANDARD, "judge": JD_MODE_JUDGE, "judge_or_standard": JD_MODE_JUDGE_OR_STANDARD}
RESAMPLE = {"residual": JD_RESAMPLE_RESIDUAL, "target_p": JD_RESAMPLE_TARGET_P}
RULES = {"sampling": JD_RULE_SAMPLING, "topk": JD_RULE_TOPK, "greedy": JD_RULE_TOPK}
VARIANTS = {"auto": JD_VARIANT_AUTO, "simt": JD_VARIANT_SIMT, "fused": JD_VARIANT_FUSED, "batched": JD_VARIANT_BATCHED}

EXPORTS = ["jd_version", "jd_status_string", "jd_workspace_bytes", "jd_create", "jd_destroy", "jd_set_head",
           "jd_verify", "jd_verify_host", "jd_last_device_status", "jd_last_launch_info", "jd_philox_uniforms",
           "jd_verify_static", "jd_set_head_fp8", "jd_selftest_timeout", "jd_stream_read_probe",
           "jd_quantize_rows_e4m3", "jd_check_workspace_guards", "jd_selftest_stale_timeout",
           "jd_debug_phase_stamps"]


class jd_config_t(C.Structure):
    _fields_ = [("max_B", C.c_int32), ("max_M", C.c_int32), ("d", C.c_int32), ("V", C.c_int32),
                ("dtype", C.c_int32), ("device", C.c_int32)]


class jd_verify_args_t(C.Structure):
    _fields_ = [("B", C.c_int32), ("M", C.c_int32), ("H", C.c_void_p), ("draft_tokens", C.c_void_p),
                ("draft_logits", C.c_void_p), ("tau", C.c_float), ("seed", C.c_uint64), ("mode", C.c_int32),
                ("resample", C.c_int32), ("variant", C.c_int32), ("rule", C.c_int32), ("top_k", C.c_int32), ("norm", C.c_int32), ("rms_eps", C.c_float),
                ("accept_len", C.c_void_p), ("next_token", C.c_void_p), ("judge_scores", C.c_void_p),
                ("p_draft", C.c_void_p), ("q_draft", C.c_void_p), ("masks", C.c_void_p),
                ("row_max", C.c_void_p), ("row_lse", C.c_void_p), ("logits_debug", C.c_void_p)]


class JdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, jd_status_string(status), status))


def library_path() -> str:
    return _LIB_PATH


def load():
    """Loads the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2501_19309_b200.build`; "
                          "there is no fallback path" % _LIB_PATH)
    lib = C.CDLL(_LIB_PATH)
    lib.jd_version.restype = C.c_int
    lib.jd_status_string.restype = C.c_char_p
    lib.jd_status_string.argtypes = [C.c_int]
    lib.jd_workspace_bytes.restype = C.c_size_t
    lib.jd_workspace_bytes.argtypes = [C.POINTER(jd_config_t)]
    lib.jd_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(jd_config_t)]
    lib.jd_destroy.argtypes = [C.c_void_p]
    lib.jd_set_head.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float]
    lib.jd_selftest_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
    lib.jd_set_head_fp8.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float]
    lib.jd_verify.argtypes = [C.c_void_p, C.POINTER(jd_verify_args_t), C.c_void_p]
    lib.jd_verify_host.argtypes = [C.c_void_p, C.POINTER(jd_verify_args_t), C.c_void_p]
    lib.jd_last_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    lib.jd_last_launch_info.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.jd_philox_uniforms.argtypes = [C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                       C.c_void_p]
    lib.jd_stream_read_probe.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.jd_verify_static.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_float,
                                     C.POINTER(jd_verify_args_t), C.c_void_p, C.c_void_p]
    lib.jd_quantize_rows_e4m3.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.jd_check_workspace_guards.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
    lib.jd_selftest_stale_timeout.argtypes = [C.c_void_p, C.c_void_p]
    lib.jd_debug_phase_stamps.argtypes = [C.c_void_p, C.c_int32]
    for name in EXPORTS:
        if name not in ("jd_version", "jd_status_string", "jd_workspace_bytes"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


# ------------------------------------------------------------------ C names, raw pointers
def jd_version() -> int:
    return load().jd_version()


def jd_status_string(status: int) -> str:
    return load().jd_status_string(int(status)).decode()


def jd_workspace_bytes(cfg: jd_config_t) -> int:
    return load().jd_workspace_bytes(C.byref(cfg))


def jd_create(cfg: jd_config_t) -> C.c_void_p:
    h = C.c_void_p()
    st = load().jd_create(C.byref(h), C.byref(cfg))
    if st != JD_OK:
        raise JdError(st, "jd_create")
    return h


def jd_destroy(h) -> None:
    load().jd_destroy(h)


def jd_set_head(h, W_ptr: int, w_judge_ptr: int, b_judge: float) -> int:
    return load().jd_set_head(h, C.c_void_p(W_ptr), C.c_void_p(w_judge_ptr), C.c_float(b_judge))


def jd_set_head_fp8(h, W8_ptr: int, w_scale_ptr: int, w_judge_ptr: int, b_judge: float) -> int:
    return load().jd_set_head_fp8(h, C.c_void_p(W8_ptr), C.c_void_p(w_scale_ptr), C.c_void_p(w_judge_ptr),
                                  C.c_float(b_judge))


def jd_verify(h, args: jd_verify_args_t, stream_ptr: int = 0) -> int:
    return load().jd_verify(h, C.byref(args), C.c_void_p(stream_ptr))


def jd_verify_host(h, args: jd_verify_args_t, stream_ptr: int = 0) -> int:
    return load().jd_verify_host(h, C.byref(args), C.c_void_p(stream_ptr))


def jd_selftest_timeout(h, spin_limit: int, stream_ptr: int = 0) -> int:
    return load().jd_selftest_timeout(h, C.c_uint32(spin_limit), C.c_void_p(stream_ptr))


def jd_debug_phase_stamps(out_ptr: int, capacity: int) -> int:
    """Copies the fused kernel's phase stamps into a host array of uint64 (stamps build only); see jd.h."""
    return load().jd_debug_phase_stamps(C.c_void_p(out_ptr), C.c_int32(capacity))


def jd_selftest_stale_timeout(h, stream_ptr: int = 0) -> int:
    return load().jd_selftest_stale_timeout(h, C.c_void_p(stream_ptr))


def jd_last_device_status(h) -> int:
    out = C.c_int(0)
    st = load().jd_last_device_status(h, C.byref(out))
    if st != JD_OK:
        raise JdError(st, "jd_last_device_status")
    return out.value


def jd_last_launch_info(h):
    v, n = C.c_int(0), C.c_int(0)
    load().jd_last_launch_info(h, C.byref(v), C.byref(n))
    return v.value, n.value


def jd_philox_uniforms(seed: int, b_ptr: int, slot_ptr: int, stream_idx_ptr: int, n: int, out_ptr: int,
                       stream_ptr: int = 0) -> int:
    return load().jd_philox_uniforms(C.c_uint64(seed), C.c_void_p(b_ptr), C.c_void_p(slot_ptr),
                                     C.c_void_p(stream_idx_ptr), C.c_int32(n), C.c_void_p(out_ptr),
                                     C.c_void_p(stream_ptr))


def jd_stream_read_probe(data_ptr: int, nbytes: int, out_ptr: int, stream_ptr: int = 0) -> int:
    """Reads nbytes at data_ptr once and XORs every 32-bit word into the word at out_ptr; see jd.h."""
    return load().jd_stream_read_probe(C.c_void_p(data_ptr), C.c_size_t(nbytes), C.c_void_p(out_ptr),
                                       C.c_void_p(stream_ptr))


def jd_quantize_rows_e4m3(H_ptr: int, rows: int, d: int, codes_ptr: int, scale_ptr: int, stream_ptr: int = 0) -> int:
    """The library's per-row E4M3 quantiser on its own (test helper); see jd.h."""
    return load().jd_quantize_rows_e4m3(C.c_void_p(H_ptr), C.c_int32(rows), C.c_int32(d), C.c_void_p(codes_ptr),
                                        C.c_void_p(scale_ptr), C.c_void_p(stream_ptr))


def jd_check_workspace_guards(h) -> int:
    """Number of damaged guard blocks between the handle's workspace regions (0 = intact)."""
    out = C.c_int32(-1)
    st = load().jd_check_workspace_guards(h, C.byref(out))
    if st != JD_OK:
        raise JdError(st, "jd_check_workspace_guards")
    return out.value


def jd_verify_static(d: int, V: int, W_ptr: int, w_judge_ptr: int, b_judge: float, args: jd_verify_args_t,
                     device_status_ptr: int = 0, stream_ptr: int = 0) -> int:
    """Handle-free verification that allocates nothing (fixed scratch inside the library); see jd.h."""
    return load().jd_verify_static(C.c_int32(d), C.c_int32(V), C.c_void_p(W_ptr), C.c_void_p(w_judge_ptr),
                                   C.c_float(b_judge), C.byref(args), C.c_void_p(device_status_ptr or None),
                                   C.c_void_p(stream_ptr))


# ------------------------------------------------------------------ tensor-level convenience
OUTPUT_NAMES = ("accept_len", "next_token", "judge_scores", "p_draft", "q_draft", "masks", "row_max", "row_lse",
                "logits_debug")


class Verifier:
    """Owns a handle; marshals torch tensors to ``jd_verify`` / ``jd_verify_host``."""

    def __init__(self, max_B: int, max_M: int, d: int, V: int, dtype: str = "bf16", device: int = 0):
        import torch
        self.torch = torch
        code = {"bf16": JD_DTYPE_BF16, "f32": JD_DTYPE_F32, "fp8": JD_DTYPE_FP8_E4M3}[dtype]
        self.cfg = jd_config_t(max_B, max_M, d, V, code, device)
        self.fp8 = dtype == "fp8"
        self.dtype = torch.float32 if dtype == "f32" else torch.bfloat16     # type of H and w_judge
        self.device = torch.device("cuda", device)
        self.h = jd_create(self.cfg)
        self._W = self._w = None

    def close(self) -> None:
        if getattr(self, "h", None) is not None:
            jd_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_head(self, W, w_judge, b_judge: float, w_scale=None) -> None:
        """W: [V, d] in the handle's dtype; for an FP8 head W holds uint8 E4M3 codes and w_scale [V]
        (float32) is required."""
        t = self.torch
        assert W.is_cuda and W.is_contiguous() and tuple(W.shape) == (self.cfg.V, self.cfg.d)
        assert w_judge.is_cuda and w_judge.dtype == self.dtype and w_judge.is_contiguous()
        self._W, self._w, self._ws = W, w_judge, w_scale         # keep the borrowed tensors alive
        if self.fp8:
            assert W.dtype == t.uint8 and w_scale is not None and w_scale.dtype == t.float32 and w_scale.is_cuda
            st = jd_set_head_fp8(self.h, W.data_ptr(), w_scale.data_ptr(), w_judge.data_ptr(), float(b_judge))
            if st != JD_OK:
                raise JdError(st, "jd_set_head_fp8")
            return
        assert W.dtype == self.dtype
        st = jd_set_head(self.h, W.data_ptr(), w_judge.data_ptr(), float(b_judge))
        if st != JD_OK:
            raise JdError(st, "jd_set_head")

    def alloc_outputs(self, B: int, M: int, debug_logits: bool = False, host: bool = False) -> dict:
        t = self.torch
        kw = dict(device="cpu", pin_memory=True) if host else dict(device=self.device)
        out = dict(accept_len=t.full((B,), -7, dtype=t.int32, **kw),
                   next_token=t.full((B,), -7, dtype=t.int32, **kw),
                   judge_scores=t.zeros((B, M), dtype=t.float32, **kw),
                   p_draft=t.zeros((B, M), dtype=t.float32, **kw),
                   q_draft=t.zeros((B, M), dtype=t.float32, **kw),
                   masks=t.zeros((B, M), dtype=t.uint8, **kw),
                   row_max=t.zeros((B, M + 1), dtype=t.float32, **kw),
                   row_lse=t.zeros((B, M + 1), dtype=t.float32, **kw))
        if debug_logits:
            out["logits_debug"] = t.zeros((B, M + 1, self.cfg.V), dtype=t.float32, **kw)
        return out

    def make_args(self, H, draft_tokens, draft_logits, tau: float, seed: int, mode="judge_or_standard",
                  resample="residual", variant="auto", out: Optional[dict] = None, host: bool = False,
                  rule="sampling", top_k: int = 1, rms_eps: Optional[float] = None):
        B, Mp1, _ = H.shape
        M = Mp1 - 1
        if out is None:
            out = self.alloc_outputs(B, M, host=host)
        a = jd_verify_args_t()
        a.B, a.M = B, M
        a.H, a.draft_tokens, a.draft_logits = H.data_ptr(), draft_tokens.data_ptr(), draft_logits.data_ptr()
        a.tau, a.seed = float(tau), int(seed)
        a.mode = MODES[mode] if isinstance(mode, str) else int(mode)
        a.resample = RESAMPLE[resample] if isinstance(resample, str) else int(resample)
        a.variant = VARIANTS[variant] if isinstance(variant, str) else int(variant)
        a.rule = RULES[rule] if isinstance(rule, str) else int(rule)
        a.top_k = 1 if rule == "greedy" else int(top_k)
        a.norm = JD_NORM_NONE if rms_eps is None else JD_NORM_RMS
        a.rms_eps = 0.0 if rms_eps is None else float(rms_eps)
        for k in OUTPUT_NAMES:
            setattr(a, k, out[k].data_ptr() if out.get(k) is not None else None)
        return a, out

    def verify(self, H, draft_tokens, draft_logits, tau: float, seed: int, mode="judge_or_standard",
               resample="residual", variant="auto", out: Optional[dict] = None, stream=None,
               rule="sampling", top_k: int = 1, rms_eps: Optional[float] = None) -> dict:
        """Enqueues one verification on ``stream`` (default: torch's current stream); returns the
        dict of output tensors (device)."""
        t = self.torch
        assert H.is_cuda and H.dtype == self.dtype and H.is_contiguous()
        assert draft_tokens.dtype == t.int32 and draft_tokens.is_contiguous() and draft_tokens.is_cuda
        assert draft_logits.dtype == t.float32 and draft_logits.is_contiguous() and draft_logits.is_cuda
        a, out = self.make_args(H, draft_tokens, draft_logits, tau, seed, mode, resample, variant, out,
                                rule=rule, top_k=top_k, rms_eps=rms_eps)
        s = stream if stream is not None else t.cuda.current_stream(self.device)
        st = jd_verify(self.h, a, s.cuda_stream)
        if st != JD_OK:
            raise JdError(st, "jd_verify")
        return out

    def verify_host(self, H, draft_tokens, draft_logits, tau: float, seed: int, mode="judge_or_standard",
                    resample="residual", variant="auto", out: Optional[dict] = None, stream=None) -> dict:
        """Host-buffer call: inputs and outputs are CPU tensors (pinned recommended); returns after
        the outputs have arrived."""
        t = self.torch
        assert not H.is_cuda and H.dtype == self.dtype and H.is_contiguous()
        assert not draft_tokens.is_cuda and draft_tokens.dtype == t.int32 and draft_tokens.is_contiguous()
        assert not draft_logits.is_cuda and draft_logits.dtype == t.float32 and draft_logits.is_contiguous()
        a, out = self.make_args(H, draft_tokens, draft_logits, tau, seed, mode, resample, variant, out, host=True)
        s = stream if stream is not None else t.cuda.current_stream(self.device)
        st = jd_verify_host(self.h, a, s.cuda_stream)
        if st != JD_OK:
            raise JdError(st, "jd_verify_host")
        return out

    def device_status(self) -> int:
        return jd_last_device_status(self.h)

    def launch_info(self):
        return jd_last_launch_info(self.h)

    def damaged_guards(self) -> int:
        return jd_check_workspace_guards(self.h)
