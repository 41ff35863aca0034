"""ctypes binding of include/stmoe.h: same names, argument marshalling only.

torch is used for device memory and stream handles; every tensor handed to a
call must live on the CUDA device (or be a host tensor where the header says
"host").  The library is loaded from the package directory and must have been
built (paper_2606_15453_b200.build.build()); there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

DTYPE = {"f32": 0, "bf16": 1, "fp8": 2}
MODE = {"off": 0, "temporal": 1, "spatial": 2, "st": 3}
FLAG_RENORM_TOPK = 1
FLAG_NO_PERSISTENT = 2
FLAG_NO_DENSE = 4
FLAG_NO_FUSED = 8
HOOK_DROP_PREFETCH, HOOK_FAIL_COPY, HOOK_DELAY_COPY_US, HOOK_CORRUPT_TAG, HOOK_HOST_WAIT_MS, HOOK_POLL_LIMIT = 1, 2, 3, 4, 5, 6


class StmoeError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32),
                ("n_shared", C.c_int32), ("hidden", C.c_int32), ("inter", C.c_int32),
                ("max_batch", C.c_int32), ("weight_dtype", C.c_int32), ("cache_slots", C.c_int64),
                ("profile_tokens", C.c_int32), ("predictor_mode", C.c_int32), ("flags", C.c_int32),
                ("prefetch_limit", C.c_int32), ("rms_eps", C.c_float), ("residual_scale", C.c_float)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "decode_steps", "runtime_steps", "routed", "predicted", "hits", "near_ties", "cache_hits",
        "cache_misses", "prefetch_issued", "prefetch_useful", "prefetch_wasted", "prefetch_dropped",
        "prefetch_resident", "h2d_bytes_demand", "h2d_bytes_prefetch")] + \
        [("transfer_ms", C.c_double), ("exposed_ms", C.c_double), ("kernel_launches", C.c_int64),
         ("timed_ffn_launches", C.c_int64), ("gate_up_ms", C.c_double), ("down_ms", C.c_double),
         ("router_ms", C.c_double), ("recovered_faults", C.c_int64)]


_lib = None


def lib():
    """Load libstmoe.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.LIB):
            raise StmoeError(f"{_build.LIB} is missing: run paper_2606_15453_b200.build.build()")
        L = C.CDLL(_build.LIB)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t
        L.stmoe_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
        L.stmoe_destroy.argtypes = [vp]
        L.stmoe_strerror.restype = C.c_char_p
        L.stmoe_strerror.argtypes = [i32]
        L.stmoe_load_router.argtypes = [vp, i32, vp]
        L.stmoe_load_experts.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, i32]
        L.stmoe_decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.stmoe_decode_token.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.stmoe_decode_token_host.argtypes = [vp, i32, vp, vp, vp, vp]
        L.stmoe_max_predicted.argtypes = [vp]
        L.stmoe_set_kernel_timing.argtypes = [vp, i32]
        L.stmoe_set_dense_min_batch.argtypes = [vp, i32]
        L.stmoe_set_prefetch_min_score.argtypes = [vp, i32]
        L.stmoe_set_onchip_staging.argtypes = [vp, i64, i64]
        L.stmoe_set_cache_policy.argtypes = [vp, i32, i32, i32]
        L.stmoe_set_predict_threshold.argtypes = [vp, i32]
        L.stmoe_set_replacement_rule.argtypes = [vp, i32]
        L.stmoe_set_copy_throttle.argtypes = [vp, i64, i32]
        L.stmoe_test_hook.argtypes = [vp, i32, i64]
        L.stmoe_selftest_bounded_wait.argtypes = [vp, i32, i32, vp]
        L.stmoe_stats.argtypes = [vp, C.POINTER(Stats)]
        L.stmoe_export_state.argtypes = [vp, vp, C.POINTER(sz)]
        L.stmoe_import_state.argtypes = [vp, vp, sz]
        L.stmoe_export_cache_tags.argtypes = [vp, vp, i64]
        L.stmoe_router_topk.argtypes = [vp, vp, i32, i32, i32, i32, i32, f32, i32, vp, vp, vp, vp, vp]
        L.stmoe_predictor_step.argtypes = [vp, i32, i32, vp, vp, vp, vp]
        L.stmoe_expert_image_bytes.restype = sz
        L.stmoe_expert_image_bytes.argtypes = [i32, i32, i32]
        L.stmoe_moe_ffn_scratch_bytes.restype = sz
        L.stmoe_moe_ffn_scratch_bytes.argtypes = [i32, i32, i32, i32]
        L.stmoe_moe_ffn.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp, sz, vp]
        L.stmoe_moe_ffn_static.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp]
        L.stmoe_expert_ffn_dense_scratch_bytes.restype = sz
        L.stmoe_expert_ffn_dense_scratch_bytes.argtypes = [i32, i32, i32]
        L.stmoe_expert_ffn_dense.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise StmoeError(f"{what}: {lib().stmoe_strerror(rc).decode()} ({rc})")


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _dev(t, dtype=None):
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t.data_ptr()


def _stream(stream):
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


class Stack:
    """Owns one stmoe_t.  Methods mirror the C entry points one to one."""

    def __init__(self, n_layers, n_experts, top_k, hidden, inter, n_shared=0, max_batch=1,
                 dtype="bf16", cache_slots=0, profile_tokens=0, mode="st", flags=0,
                 prefetch_limit=0, rms_eps=1e-6, residual_scale=0.1):
        self.cfg = Config(n_layers, n_experts, top_k, n_shared, hidden, inter, max_batch,
                          DTYPE[dtype], cache_slots, profile_tokens, MODE[mode], flags,
                          prefetch_limit, rms_eps, residual_scale)
        self._h = C.c_void_p()
        _check(lib().stmoe_create(C.byref(self.cfg), C.byref(self._h)), "stmoe_create")
        self.max_pred = lib().stmoe_max_predicted(self._h)
        self.dtype = dtype

    @classmethod
    def from_config(cls, cfg, max_batch=1, **kw):
        """cfg: an object with the fields of datagen.StackConfig."""
        args = dict(n_layers=cfg.n_layers, n_experts=cfg.n_experts, top_k=cfg.top_k,
                    hidden=cfg.hidden, inter=cfg.inter, n_shared=cfg.n_shared,
                    max_batch=max_batch, dtype=cfg.dtype, cache_slots=cfg.cache_slots,
                    profile_tokens=cfg.profile_tokens, rms_eps=cfg.rms_eps,
                    residual_scale=cfg.residual_scale)
        args.update(kw)
        return cls(**args)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().stmoe_destroy(self._h)
            self._h = C.c_void_p()

    __del__ = close

    def load_router(self, layer: int, w: torch.Tensor) -> None:
        _check(lib().stmoe_load_router(self._h, layer, _ptr(w)), "stmoe_load_router")

    def load_experts(self, layer, first_expert, gate, up, down, scales=None, shared=False) -> None:
        """gate/up [n][I][H], down [n][H][I] (or 2-D for one expert), host or device.  The call copies
        at once and does not know torch's streams: synchronise the stream that produced a device
        source before calling."""
        count = 1 if gate.dim() == 2 else gate.shape[0]
        _check(lib().stmoe_load_experts(self._h, layer, first_expert, count, _ptr(gate), _ptr(up),
                                        _ptr(down), _ptr(scales), int(shared)), "stmoe_load_experts")

    def decode_step(self, layer, h_in, h_out, routed_ids=None, routed_w=None, predicted_ids=None,
                    n_predicted=None, flags=None, stream=None) -> None:
        b = h_in.shape[0]
        _check(lib().stmoe_decode_step(self._h, layer, b, _dev(h_in, torch.float32),
                                       _dev(h_out, torch.float32), _ptr(routed_ids), _ptr(routed_w),
                                       _ptr(predicted_ids), _ptr(n_predicted), _ptr(flags),
                                       _stream(stream)), "stmoe_decode_step")

    def decode_token(self, h_in, h_out, routed_ids=None, routed_w=None, predicted_ids=None,
                     n_predicted=None, flags=None, stream=None) -> None:
        b = h_in.shape[0]
        _check(lib().stmoe_decode_token(self._h, b, _dev(h_in, torch.float32),
                                        _dev(h_out, torch.float32), _ptr(routed_ids), _ptr(routed_w),
                                        _ptr(predicted_ids), _ptr(n_predicted), _ptr(flags),
                                        _stream(stream)), "stmoe_decode_token")

    def decode_token_host(self, h_in, h_out, routed_ids=None, stream=None) -> None:
        """h_in / h_out / routed_ids: CPU tensors (pinned for full copy speed); returns when done."""
        assert not h_in.is_cuda and not h_out.is_cuda and h_in.is_contiguous() and h_out.is_contiguous()
        assert h_in.dtype == torch.float32 and h_out.dtype == torch.float32
        assert routed_ids is None or (not routed_ids.is_cuda and routed_ids.dtype == torch.int32)
        _check(lib().stmoe_decode_token_host(self._h, h_in.shape[0], h_in.data_ptr(), h_out.data_ptr(),
                                             _ptr(routed_ids), _stream(stream)), "stmoe_decode_token_host")

    def predictor_step(self, layer, routed_ids, predicted_ids=None, n_predicted=None,
                       stream=None) -> None:
        _check(lib().stmoe_predictor_step(self._h, layer, routed_ids.shape[0],
                                          _dev(routed_ids, torch.int32), _ptr(predicted_ids),
                                          _ptr(n_predicted), _stream(stream)), "stmoe_predictor_step")

    def set_kernel_timing(self, on: bool) -> None:
        _check(lib().stmoe_set_kernel_timing(self._h, int(on)), "stmoe_set_kernel_timing")

    def set_prefetch_min_score(self, min_score: int) -> None:
        _check(lib().stmoe_set_prefetch_min_score(self._h, int(min_score)), "stmoe_set_prefetch_min_score")

    def set_onchip_staging(self, known_bytes: int, predicted_bytes: int) -> None:
        _check(lib().stmoe_set_onchip_staging(self._h, int(known_bytes), int(predicted_bytes)),
               "stmoe_set_onchip_staging")

    def set_predict_threshold(self, threshold: int) -> None:
        _check(lib().stmoe_set_predict_threshold(self._h, int(threshold)), "stmoe_set_predict_threshold")

    def set_replacement_rule(self, live_counts: bool) -> None:
        _check(lib().stmoe_set_replacement_rule(self._h, int(bool(live_counts))), "stmoe_set_replacement_rule")

    def set_cache_policy(self, history_window: int, by_turn: bool, prefetch_floor: int = -1) -> None:
        _check(lib().stmoe_set_cache_policy(self._h, int(history_window), int(by_turn), int(prefetch_floor)),
               "stmoe_set_cache_policy")

    def set_copy_throttle(self, chunk_bytes: int, gap_us: int) -> None:
        _check(lib().stmoe_set_copy_throttle(self._h, int(chunk_bytes), int(gap_us)), "stmoe_set_copy_throttle")

    def test_hook(self, what: int, value: int) -> None:
        _check(lib().stmoe_test_hook(self._h, int(what), int(value)), "stmoe_test_hook")

    def selftest_bounded_wait(self, which: int, poll_limit: int = 4096, stream=None) -> None:
        _check(lib().stmoe_selftest_bounded_wait(self._h, int(which), int(poll_limit), _stream(stream)),
               "stmoe_selftest_bounded_wait")

    def set_dense_min_batch(self, min_batch: int) -> None:
        _check(lib().stmoe_set_dense_min_batch(self._h, int(min_batch)), "stmoe_set_dense_min_batch")

    def stats(self) -> dict:
        st = Stats()
        _check(lib().stmoe_stats(self._h, C.byref(st)), "stmoe_stats")
        return {n: getattr(st, n) for n, _ in Stats._fields_}

    def export_state(self) -> bytes:
        n = C.c_size_t(0)
        _check(lib().stmoe_export_state(self._h, None, C.byref(n)), "stmoe_export_state")
        buf = C.create_string_buffer(n.value)
        _check(lib().stmoe_export_state(self._h, buf, C.byref(n)), "stmoe_export_state")
        return buf.raw[:n.value]

    def import_state(self, blob: bytes) -> None:
        _check(lib().stmoe_import_state(self._h, blob, len(blob)), "stmoe_import_state")

    def export_cache_tags(self) -> torch.Tensor:
        t = torch.empty(self.cfg.cache_slots, dtype=torch.int32)
        _check(lib().stmoe_export_cache_tags(self._h, t.data_ptr(), t.numel()), "stmoe_export_cache_tags")
        return t


def router_topk(h, w_router, top_k, rms_eps=1e-6, renorm=False, stream=None):
    """Gating network for h [B][H] (fp32) and w_router [E][H] (fp32 or bf16), on the GPU.
    Returns dict(logits [B][E], inv_rms [B], ids [B][K], w [B][K], flags [B])."""
    B, H = h.shape
    E = w_router.shape[0]
    wdt = 0 if w_router.dtype == torch.float32 else 1
    buf = torch.empty(B * E + B, dtype=torch.float32, device=h.device)
    ids = torch.empty(B, top_k, dtype=torch.int32, device=h.device)
    w = torch.empty(B, top_k, dtype=torch.float32, device=h.device)
    flags = torch.empty(B, dtype=torch.int32, device=h.device)
    _check(lib().stmoe_router_topk(_dev(h, torch.float32), _dev(w_router), wdt, B, E, H, top_k,
                                   rms_eps, int(renorm), _dev(buf), _dev(ids), _dev(w), _dev(flags),
                                   _stream(stream)), "stmoe_router_topk")
    return dict(logits=buf[:B * E].view(B, E), inv_rms=buf[B * E:], ids=ids, w=w, flags=flags)


def expert_image_bytes(hidden, inter, dtype) -> int:
    return lib().stmoe_expert_image_bytes(hidden, inter, DTYPE[dtype])


def moe_ffn_scratch_bytes(batch, top_k, hidden, inter) -> int:
    return lib().stmoe_moe_ffn_scratch_bytes(batch, top_k, hidden, inter)


def moe_ffn(h, inv_rms, ids, w, experts, dtype, n_experts, hidden, inter, residual_scale, h_out,
            scratch, stream=None, entry="stmoe_moe_ffn"):
    """Routed SwiGLU FFN + weighted sum + residual for given routing (all tensors on the GPU).
    experts: uint8 tensor of n_experts expert images."""
    B, K = ids.shape
    fn = getattr(lib(), entry)
    _check(fn(_dev(h, torch.float32), _ptr(inv_rms), _dev(ids, torch.int32), _dev(w, torch.float32),
              _dev(experts), DTYPE[dtype], B, n_experts, K, hidden, inter, residual_scale,
              _dev(h_out, torch.float32), _dev(scratch), scratch.numel() * scratch.element_size(),
              _stream(stream)), entry)
    return h_out


def moe_ffn_static(h, inv_rms, ids, w, experts, dtype, n_experts, hidden, inter, residual_scale, h_out,
                   stream=None):
    """stmoe_moe_ffn_static: the same computation as moe_ffn for callers that must not allocate
    device memory; scratch is an 8 MiB area inside the library, shared by every call on the
    device (order calls that could overlap).  Raises StmoeError when the problem needs more."""
    B, K = ids.shape
    _check(lib().stmoe_moe_ffn_static(_dev(h, torch.float32), _ptr(inv_rms), _dev(ids, torch.int32),
                                      _dev(w, torch.float32), _dev(experts), DTYPE[dtype], B, n_experts, K,
                                      hidden, inter, residual_scale, _dev(h_out, torch.float32),
                                      _stream(stream)), "stmoe_moe_ffn_static")
    return h_out


def expert_ffn_dense(h, inv_rms, image, hidden, inter, stream=None):
    """stmoe_expert_ffn_dense: one bf16 expert's SwiGLU FFN for the m <= 64 tokens in h [m][hidden]
    on the tensor cores.  Returns (y [m][hidden] fp32, flags uint32 tensor; non-zero = a bounded
    wait inside a kernel ran out)."""
    m = h.shape[0]
    n = lib().stmoe_expert_ffn_dense_scratch_bytes(m, hidden, inter)
    scratch = torch.empty(max(n, 256), dtype=torch.uint8, device=h.device)
    y = torch.empty(m, hidden, dtype=torch.float32, device=h.device)
    flags = torch.zeros(1, dtype=torch.int32, device=h.device)
    _check(lib().stmoe_expert_ffn_dense(_dev(h, torch.float32), _ptr(inv_rms), _dev(image), m, hidden, inter,
                                        _dev(y), _dev(flags), _dev(scratch), scratch.numel(), _stream(stream)),
           "stmoe_expert_ffn_dense")
    return y, flags
