"""Python binding of the B200 flash-attention C-ABI library (include/attn.h).

Argument marshalling only: every step of the hot path runs in the CUDA kernels
of libattn_b200.so.  The functions carry the names of the C entry points and
take torch CUDA tensors (or raw device addresses as int) in the layout the
header states: BF16 [B,H,N,d] contiguous, FP32 [B,H,N] for lse and delta.

There is no CPU fallback: importing this package without the compiled library
(and without nvcc to build it) raises.
"""
import ctypes as C
import os

from . import build as _build

__all__ = ["AttnError", "attn_fwd", "attn_fwd_count_ones", "attn_fwd_o_f32", "attn_bwd_delta_f32", "attn_quantize_v_e4m3", "attn_fwd_fp8pv", "attn_fwd_pbar_format", "attn_bwd", "attn_bwd_stage", "attn_bwd_static", "attn_fwd_gqa", "attn_bwd_gqa", "attn_fwd_padded", "attn_bwd_padded", "attn_fwd_varlen", "attn_bwd_varlen", "attn_fwd_packed", "attn_bwd_packed", "attn_packed_workspace_bytes", "attn_bwd_preprocess", "attn_bwd_delta_dp", "attn_bwd_workspace_bytes",
           "attn_get_tiles", "attn_set_mitigation", "attn_get_mitigation", "attn_set_guard_max_shift", "attn_get_guard_max_shift", "attn_last_device_status", "attn_selftest_wait_timeout",
           "attn_strerror", "lib", "LIB_PATH", "EXPORTS"]

LIB_PATH = _build.LIB
EXPORTS = ("attn_fwd", "attn_fwd_count_ones", "attn_fwd_o_f32", "attn_bwd_delta_f32", "attn_quantize_v_e4m3", "attn_fwd_fp8pv", "attn_fwd_pbar_format", "attn_bwd", "attn_bwd_stage", "attn_bwd_static", "attn_fwd_gqa", "attn_bwd_gqa", "attn_fwd_padded", "attn_bwd_padded", "attn_fwd_varlen", "attn_bwd_varlen", "attn_fwd_packed", "attn_bwd_packed", "attn_packed_workspace_bytes", "attn_bwd_preprocess", "attn_bwd_delta_dp", "attn_bwd_workspace_bytes", "attn_get_tiles",
           "attn_set_mitigation", "attn_get_mitigation", "attn_set_guard_max_shift", "attn_get_guard_max_shift", "attn_last_device_status", "attn_selftest_wait_timeout", "attn_strerror")


class AttnError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {attn_strerror(code)} (code {int(code)})")


def _load():
    if not os.path.exists(LIB_PATH):
        _build.build()                      # raises if nvcc is missing or the build fails
    L = C.CDLL(LIB_PATH)
    if not all(hasattr(L, n) for n in EXPORTS):     # a library left over from older sources: rebuild, load the new file
        _build.build(force=True)
        L = C.CDLL(LIB_PATH)
    vp, fp, i, f, sz = C.c_void_p, C.c_void_p, C.c_int, C.c_float, C.c_size_t
    L.attn_fwd.restype = i
    L.attn_fwd.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, i, f, i, vp]
    L.attn_fwd_count_ones.restype = i
    L.attn_fwd_count_ones.argtypes = [vp, vp, vp, vp, fp, vp, i, i, i, i, i, f, i, vp]
    L.attn_fwd_pbar_format.restype = i
    L.attn_fwd_pbar_format.argtypes = [vp, vp, vp, vp, fp, vp, i, i, i, i, i, f, i, i, vp]
    L.attn_bwd_delta_dp.restype = i
    L.attn_bwd_delta_dp.argtypes = [vp, vp, vp, vp, fp, fp, i, i, i, i, i, C.c_float, vp]
    L.attn_fwd_o_f32.restype = i
    L.attn_fwd_o_f32.argtypes = [vp, vp, vp, vp, fp, fp, i, i, i, i, i, f, i, vp]
    L.attn_bwd_delta_f32.restype = i
    L.attn_bwd_delta_f32.argtypes = [fp, vp, fp, i, i, i, i, vp]
    L.attn_packed_workspace_bytes.restype = sz
    L.attn_packed_workspace_bytes.argtypes = [i, i, i, i, i, i]
    L.attn_fwd_packed.restype = i
    L.attn_fwd_packed.argtypes = [vp, vp, vp, vp, fp, vp, vp, sz, i, i, i, i, i, i, i, f, i, vp]
    L.attn_bwd_packed.restype = i
    L.attn_bwd_packed.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, vp, vp, sz, i, i, i, i, i, i, i, f, i, vp]
    L.attn_quantize_v_e4m3.restype = i
    L.attn_quantize_v_e4m3.argtypes = [vp, vp, i, i, i, i, f, vp]
    L.attn_fwd_fp8pv.restype = i
    L.attn_fwd_fp8pv.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, i, f, i, f, vp]
    L.attn_bwd_preprocess.restype = i
    L.attn_bwd_preprocess.argtypes = [vp, vp, fp, i, i, i, i, vp]
    L.attn_bwd.restype = i
    L.attn_bwd.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, vp, sz, i, i, i, i, i, f, i, vp]
    L.attn_bwd_stage.restype = i
    L.attn_bwd_stage.argtypes = [i] + L.attn_bwd.argtypes
    L.attn_bwd_static.restype = i
    L.attn_bwd_static.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, i, i, i, i, i, f, i, vp]
    L.attn_fwd_gqa.restype = i
    L.attn_fwd_gqa.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, i, i, f, i, vp]
    L.attn_bwd_gqa.restype = i
    L.attn_bwd_gqa.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, vp, sz, i, i, i, i, i, i, f, i, vp]
    L.attn_fwd_padded.restype = i
    L.attn_fwd_padded.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, i, i, i, f, i, vp]
    L.attn_bwd_padded.restype = i
    L.attn_bwd_padded.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, vp, sz, i, i, i, i, i, i, i, f, i, vp]
    L.attn_fwd_varlen.restype = i
    L.attn_fwd_varlen.argtypes = [vp, vp, vp, vp, fp, vp, i, i, i, i, i, i, f, i, vp]
    L.attn_bwd_varlen.restype = i
    L.attn_bwd_varlen.argtypes = [vp, vp, vp, vp, vp, fp, vp, vp, vp, fp, vp, sz, vp, i, i, i, i, i, i, f, i, vp]
    L.attn_bwd_workspace_bytes.restype = sz
    L.attn_bwd_workspace_bytes.argtypes = [i, i, i, i]
    L.attn_get_tiles.restype = i
    L.attn_get_tiles.argtypes = [i, C.POINTER(i), C.POINTER(i)]
    L.attn_set_guard_max_shift.restype = i
    L.attn_set_guard_max_shift.argtypes = [f]
    L.attn_get_guard_max_shift.restype = f
    L.attn_get_guard_max_shift.argtypes = []
    L.attn_set_mitigation.restype = i
    L.attn_set_mitigation.argtypes = [f, f]
    L.attn_get_mitigation.restype = i
    L.attn_get_mitigation.argtypes = [C.POINTER(f), C.POINTER(f)]
    L.attn_last_device_status.restype = i
    L.attn_last_device_status.argtypes = [vp]
    L.attn_selftest_wait_timeout.restype = i
    L.attn_selftest_wait_timeout.argtypes = [vp]
    L.attn_strerror.restype = C.c_char_p
    L.attn_strerror.argtypes = [i]
    return L


lib = _load()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(code, where):
    if code != 0:
        raise AttnError(code, where)


def attn_strerror(code):
    return lib.attn_strerror(int(code)).decode()


def attn_fwd(q, k, v, o, lse, B, H, N, d, causal, scale, mode, stream=None):
    _check(lib.attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, N, d, int(bool(causal)),
                        float(scale), int(mode), _stream(stream)), "attn_fwd")


def attn_fwd_count_ones(q, k, v, o, lse, ones, B, H, N, d, causal, scale, mode, stream=None):
    _check(lib.attn_fwd_count_ones(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(ones), B, H, N, d,
                                   int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_fwd_count_ones")


def attn_fwd_pbar_format(q, k, v, o, lse, ones, B, H, N, d, causal, scale, mode, pbar_format, stream=None):
    _check(lib.attn_fwd_pbar_format(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(ones), B, H, N, d,
                                    int(bool(causal)), float(scale), int(mode), int(pbar_format), _stream(stream)),
           "attn_fwd_pbar_format")


def attn_bwd_delta_dp(q, k, v, dO, lse, delta, B, H, N, d, causal, scale, stream=None):
    _check(lib.attn_bwd_delta_dp(_ptr(q), _ptr(k), _ptr(v), _ptr(dO), _ptr(lse), _ptr(delta), B, H, N, d,
                                 int(bool(causal)), float(scale), _stream(stream)), "attn_bwd_delta_dp")


def attn_fwd_o_f32(q, k, v, o, lse, o_f32, B, H, N, d, causal, scale, mode, stream=None):
    _check(lib.attn_fwd_o_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(o_f32), B, H, N, d,
                              int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_fwd_o_f32")


def attn_bwd_delta_f32(o_f32, dO, delta, B, H, N, d, stream=None):
    _check(lib.attn_bwd_delta_f32(_ptr(o_f32), _ptr(dO), _ptr(delta), B, H, N, d, _stream(stream)),
           "attn_bwd_delta_f32")


def attn_quantize_v_e4m3(v, v_t_e4m3, B, H, N, d, v_scale=1.0, stream=None):
    _check(lib.attn_quantize_v_e4m3(_ptr(v), _ptr(v_t_e4m3), B, H, N, d, float(v_scale), _stream(stream)),
           "attn_quantize_v_e4m3")


def attn_fwd_fp8pv(q, k, v_t_e4m3, o, lse, B, H, N, d, causal, scale, mode=0, v_descale=1.0, stream=None):
    _check(lib.attn_fwd_fp8pv(_ptr(q), _ptr(k), _ptr(v_t_e4m3), _ptr(o), _ptr(lse), B, H, N, d, int(bool(causal)),
                              float(scale), int(mode), float(v_descale), _stream(stream)), "attn_fwd_fp8pv")


def attn_bwd_preprocess(o, dO, delta, B, H, N, d, stream=None):
    _check(lib.attn_bwd_preprocess(_ptr(o), _ptr(dO), _ptr(delta), B, H, N, d, _stream(stream)),
           "attn_bwd_preprocess")


def attn_bwd(q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
             B, H, N, d, causal, scale, mode, stream=None):
    _check(lib.attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv),
                        _ptr(delta), _ptr(workspace), int(workspace_bytes), B, H, N, d, int(bool(causal)),
                        float(scale), int(mode), _stream(stream)), "attn_bwd")


def attn_bwd_stage(stage, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
                   B, H, N, d, causal, scale, mode, stream=None):
    _check(lib.attn_bwd_stage(int(stage), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq),
                              _ptr(dk), _ptr(dv), _ptr(delta), _ptr(workspace), int(workspace_bytes), B, H, N, d,
                              int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_bwd_stage")


def attn_bwd_static(q, k, v, o, dO, lse, dq, dk, dv, delta, B, H, N, d, causal, scale, mode, stream=None):
    """attn_bwd for callers that cannot allocate device memory where they call it: the FP32 dQ
    accumulator is a 32 MiB array built into the library instead of a `workspace` argument
    (so B*H*N*d <= 8,388,608).  All calls on a device share that array: do not let two of them
    overlap on the GPU.  Make the first call on a device outside any stream capture."""
    _check(lib.attn_bwd_static(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk),
                               _ptr(dv), _ptr(delta), B, H, N, d, int(bool(causal)), float(scale), int(mode),
                               _stream(stream)), "attn_bwd_static")


def attn_fwd_gqa(q, k, v, o, lse, B, H, H_kv, N, d, causal, scale, mode=0, stream=None):
    _check(lib.attn_fwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, H_kv, N, d, int(bool(causal)),
                            float(scale), int(mode), _stream(stream)), "attn_fwd_gqa")


def attn_bwd_gqa(q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes, B, H, H_kv, N, d, causal, scale,
                 mode=0, stream=None):
    _check(lib.attn_bwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv),
                            _ptr(delta), _ptr(workspace), int(workspace_bytes), B, H, H_kv, N, d, int(bool(causal)),
                            float(scale), int(mode), _stream(stream)), "attn_bwd_gqa")


def attn_fwd_padded(q, k, v, o, lse, B, H, H_kv, N, seqlen, d, causal, scale, mode=0, stream=None):
    _check(lib.attn_fwd_padded(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, H_kv, N, seqlen, d,
                               int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_fwd_padded")


def attn_bwd_padded(q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes, B, H, H_kv, N, seqlen, d,
                    causal, scale, mode=0, stream=None):
    _check(lib.attn_bwd_padded(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv),
                               _ptr(delta), _ptr(workspace), int(workspace_bytes), B, H, H_kv, N, seqlen, d,
                               int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_bwd_padded")


def attn_fwd_varlen(q, k, v, o, lse, seqlens, B, H, H_kv, N, d, causal, scale, mode=0, stream=None):
    _check(lib.attn_fwd_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(seqlens), B, H, H_kv, N, d,
                               int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_fwd_varlen")


def attn_bwd_varlen(q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes, seqlens, B, H, H_kv, N, d,
                    causal, scale, mode=0, stream=None):
    _check(lib.attn_bwd_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv),
                               _ptr(delta), _ptr(workspace), int(workspace_bytes), _ptr(seqlens), B, H, H_kv, N, d,
                               int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_bwd_varlen")


def attn_packed_workspace_bytes(B, H, H_kv, N_max, d, backward):
    return int(lib.attn_packed_workspace_bytes(B, H, H_kv, N_max, d, int(bool(backward))))


def attn_fwd_packed(q, k, v, o, lse, cu_seqlens, workspace, workspace_bytes, B, H, H_kv, T, N_max, d, causal, scale,
                    mode=0, stream=None):
    _check(lib.attn_fwd_packed(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens), _ptr(workspace),
                               int(workspace_bytes), B, H, H_kv, T, N_max, d, int(bool(causal)), float(scale), int(mode),
                               _stream(stream)), "attn_fwd_packed")


def attn_bwd_packed(q, k, v, o, dO, lse, dq, dk, dv, delta, cu_seqlens, workspace, workspace_bytes, B, H, H_kv, T, N_max,
                    d, causal, scale, mode=0, stream=None):
    _check(lib.attn_bwd_packed(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(dO), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv),
                               _ptr(delta), _ptr(cu_seqlens), _ptr(workspace), int(workspace_bytes), B, H, H_kv, T, N_max,
                               d, int(bool(causal)), float(scale), int(mode), _stream(stream)), "attn_bwd_packed")


def attn_bwd_workspace_bytes(B, H, N, d):
    return int(lib.attn_bwd_workspace_bytes(B, H, N, d))


def attn_get_tiles(d):
    br, bc = C.c_int(0), C.c_int(0)
    _check(lib.attn_get_tiles(int(d), C.byref(br), C.byref(bc)), "attn_get_tiles")
    return br.value, bc.value


def attn_set_mitigation(beta, eps):
    _check(lib.attn_set_mitigation(float(beta), float(eps)), "attn_set_mitigation")


def attn_set_guard_max_shift(max_shift):
    _check(lib.attn_set_guard_max_shift(float(max_shift)), "attn_set_guard_max_shift")


def attn_get_guard_max_shift():
    return float(lib.attn_get_guard_max_shift())


def attn_get_mitigation():
    b, e = C.c_float(0), C.c_float(0)
    _check(lib.attn_get_mitigation(C.byref(b), C.byref(e)), "attn_get_mitigation")
    return b.value, e.value


def attn_last_device_status(stream=None):
    """Call after synchronising. Returns 0 or the ATTN_ERR_TIMEOUT code (does not raise)."""
    return int(lib.attn_last_device_status(_stream(stream) if stream is not None else None))


def attn_selftest_wait_timeout(stream=None):
    """Enqueue the kernel whose bounded waits run out by construction (about a millisecond); see attn.h."""
    _check(lib.attn_selftest_wait_timeout(_stream(stream) if stream is not None else None), "attn_selftest_wait_timeout")
