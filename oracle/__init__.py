"""ctypes access to the CPU oracle (oracle/stmoe_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stmoe_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_stmoe.so")

DTYPE_CODE = {"f32": 0, "bf16": 1, "fp8": 2}
MODE = {"off": 0, "temporal": 1, "spatial": 2, "st": 3}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP on the row loops of the FFN only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O3", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
        L.orc_bf16_to_f32.restype = f32
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_e4m3_to_f32.restype = f32
        L.orc_e4m3_to_f32.argtypes = [C.c_uint8]
        L.orc_get_threads.restype = C.c_int
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_rmsnorm.argtypes = [vp, i32, f32, vp]
        L.orc_router_logits.argtypes = [vp, vp, i32, i32, i32, vp]
        L.orc_softmax.argtypes = [vp, i32, vp]
        L.orc_topk.argtypes = [vp, i32, i32, vp, vp]
        L.orc_route.argtypes = [vp, vp, i32, i32, i32, i32, f32, i32, vp, vp, vp, vp, vp]
        L.orc_expert_ffn.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, i32, vp]
        L.orc_combine.argtypes = [vp, i32, vp, i32, vp, vp, i32, f32, vp]
        L.orc_co_accumulate.argtypes = [vp, i32, vp, i32, vp, i32]
        L.orc_cct_build.argtypes = [vp, i32, i32, vp, vp]
        L.orc_predict.restype = C.c_int
        L.orc_predict.argtypes = [i32, i32, vp, i32, vp, vp, vp, vp, vp, vp]
        L.orc_update.argtypes = [i32, i32, vp, i32, vp, i32, vp, vp]
        L.orc_update_rule.argtypes = [i32, i32, vp, i32, vp, i32, vp, vp, vp]
        L.orc_pred_set_replacement.argtypes = [vp, i32]
        L.orc_pred_create.restype = vp
        L.orc_pred_create.argtypes = [i32] * 6
        L.orc_pred_destroy.argtypes = [vp]
        L.orc_pred_set_threshold.argtypes = [vp, i32]
        L.orc_predict_thr.restype = C.c_int
        L.orc_predict_thr.argtypes = [i32, i32, vp, i32, vp, vp, vp, i32, vp, vp, vp]
        L.orc_pred_max_pred.restype = C.c_int
        L.orc_pred_max_pred.argtypes = [vp]
        L.orc_pred_step.restype = C.c_int
        L.orc_pred_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.orc_pred_stats.argtypes = [vp, vp]
        L.orc_pred_state_bytes.restype = C.c_size_t
        L.orc_pred_state_bytes.argtypes = [vp]
        L.orc_pred_export.restype = C.c_size_t
        L.orc_pred_export.argtypes = [vp, vp]
        L.orc_cache_create.restype = vp
        L.orc_cache_create.argtypes = [i64, i32, i32]
        L.orc_cache_create2.restype = vp
        L.orc_cache_create2.argtypes = [i64, i32, i32, i32, i32, i32]
        L.orc_cache_destroy.argtypes = [vp]
        L.orc_cache_step.restype = C.c_int
        L.orc_cache_step.argtypes = [vp, i32, vp, i32, i32, vp, i32, i32, vp, vp, vp]
        L.orc_cache_stats.argtypes = [vp, vp]
        L.orc_cache_tags.argtypes = [vp, vp]
        _lib = L
    return _lib


def _p(a):
    """Raw pointer of a contiguous numpy array / CPU torch tensor (or None)."""
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        assert a.device.type == "cpu" and a.is_contiguous()
        return a.data_ptr()
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


# ---------------------------------------------------------------- Section 2
def rmsnorm(h: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.float32)
    x = np.empty_like(h)
    lib().orc_rmsnorm(_p(h), h.size, eps, _p(x))
    return x


def router_logits(x: np.ndarray, Wr: torch.Tensor, dtype: str) -> np.ndarray:
    E, H = Wr.shape
    x = np.ascontiguousarray(x, dtype=np.float32)
    z = np.empty(E, dtype=np.float32)
    lib().orc_router_logits(_p(x), _p(Wr), DTYPE_CODE[dtype], E, H, _p(z))
    return z


def softmax(z: np.ndarray) -> np.ndarray:
    z = np.ascontiguousarray(z, dtype=np.float32)
    s = np.empty_like(z)
    lib().orc_softmax(_p(z), z.size, _p(s))
    return s


def topk(z: np.ndarray, K: int):
    z = np.ascontiguousarray(z, dtype=np.float32)
    ids = np.empty(K, dtype=np.int32)
    gap = np.empty(1, dtype=np.float32)
    lib().orc_topk(_p(z), z.size, K, _p(ids), _p(gap))
    return ids, float(gap[0])


def route(h: np.ndarray, Wr: torch.Tensor, dtype: str, K: int, eps: float = 1e-6,
          renorm: bool = False):
    """One token: returns dict(x, z, ids, w, near_tie)."""
    E, H = Wr.shape
    h = np.ascontiguousarray(h, dtype=np.float32)
    x = np.empty(H, dtype=np.float32)
    z = np.empty(E, dtype=np.float32)
    ids = np.empty(K, dtype=np.int32)
    w = np.empty(K, dtype=np.float32)
    tie = np.zeros(1, dtype=np.int32)
    lib().orc_route(_p(h), _p(Wr), DTYPE_CODE[dtype], E, H, K, eps, int(renorm), _p(x), _p(z),
                    _p(ids), _p(w), _p(tie))
    return dict(x=x, z=z, ids=ids, w=w, near_tie=int(tie[0]))


def expert_ffn(x: np.ndarray, wts: dict, dtype: str) -> np.ndarray:
    """wts: gate [I][H], up [I][H], down [H][I] (+ *_scale for fp8), CPU tensors."""
    I, H = wts["gate"].shape
    x = np.ascontiguousarray(x, dtype=np.float32)
    y = np.empty(H, dtype=np.float32)
    lib().orc_expert_ffn(_p(x), H, I, _p(wts["gate"]), _p(wts["up"]), _p(wts["down"]),
                         _p(wts.get("gate_scale")), _p(wts.get("up_scale")),
                         _p(wts.get("down_scale")), DTYPE_CODE[dtype], _p(y))
    return y


def combine(h, ys, yk, w, residual_scale: float) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.float32)
    H = h.size
    ys = np.ascontiguousarray(ys, dtype=np.float32).reshape(-1, H) if ys is not None and len(ys) \
        else np.zeros((0, H), dtype=np.float32)
    yk = np.ascontiguousarray(yk, dtype=np.float32).reshape(-1, H)
    w = np.ascontiguousarray(w, dtype=np.float32)
    out = np.empty(H, dtype=np.float32)
    lib().orc_combine(_p(h), H, _p(ys), ys.shape[0], _p(yk), _p(w), yk.shape[0], residual_scale,
                      _p(out))
    return out


# ------------------------------------------------------------- Algorithms 1-3
def co_accumulate(Co: np.ndarray, Ei, Fi) -> None:
    assert Co.dtype == np.uint32 and Co.flags["C_CONTIGUOUS"]
    Ei, Fi = _i32(Ei), _i32(Fi)
    lib().orc_co_accumulate(_p(Co), Co.shape[0], _p(Ei), Ei.size, _p(Fi), Fi.size)


def cct_build(Co: np.ndarray, K: int):
    E = Co.shape[0]
    ids = np.empty((E, K), dtype=np.uint8)
    conf = np.empty((E, K), dtype=np.uint8)
    lib().orc_cct_build(_p(np.ascontiguousarray(Co, dtype=np.uint32)), E, K, _p(ids), _p(conf))
    return ids, conf


def predict(E: int, K: int, Ei, cct_id, cct_conf, ht, threshold: int = 2):
    """Returns (score [E] per Eq. 1, literal-listing score [E], set mask [E])."""
    Ei = _i32(Ei)
    score = np.empty(E, dtype=np.int32)
    lit = np.empty(E, dtype=np.int32)
    mask = np.empty(E, dtype=np.uint8)
    htp = None if ht is None else np.ascontiguousarray(np.asarray(ht, dtype=np.int16))
    rc = lib().orc_predict_thr(E, K, _p(Ei), Ei.size, _p(cct_id), _p(cct_conf), _p(htp), threshold,
                               _p(score), _p(lit), _p(mask))
    if rc < 0:
        raise AssertionError("Eq. 1 and the literal listing of Algorithm 2 disagree")
    return score, lit, mask


def update(E: int, K: int, Ei, Fj, cct_id: np.ndarray, cct_conf: np.ndarray, co: np.ndarray | None = None) -> None:
    """Algorithm 3 on one layer pair.  co = None: a replaced slot takes the lowest routed id the row
    does not hold; co = the pair's [E][E] counts (already holding this step's pairs): the routed id
    with the largest count in the row."""
    Ei, Fj = _i32(Ei), _i32(Fj)
    assert cct_id.dtype == np.uint8 and cct_conf.dtype == np.uint8
    if co is None:
        lib().orc_update(E, K, _p(Ei), Ei.size, _p(Fj), Fj.size, _p(cct_id), _p(cct_conf))
    else:
        assert co.dtype == np.uint32 and co.shape == (E, E) and co.flags.c_contiguous
        lib().orc_update_rule(E, K, _p(Ei), Ei.size, _p(Fj), Fj.size, _p(cct_id), _p(cct_conf), _p(co))


class Predictor:
    """Whole-stack predictor state machine (profiling, build, verify/update, predict)."""

    def __init__(self, L, E, K, B=1, P=0, mode="st", threshold=2, live_counts=False):
        self.L, self.E, self.K, self.B, self.P = L, E, K, B, P
        self._h = lib().orc_pred_create(L, E, K, B, P, MODE[mode])
        if not self._h:
            raise ValueError("bad predictor shape")
        lib().orc_pred_set_threshold(self._h, threshold)
        lib().orc_pred_set_replacement(self._h, int(live_counts))
        self.max_pred = lib().orc_pred_max_pred(self._h)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_pred_destroy(self._h)
            self._h = None

    def step(self, layer: int, routed) -> dict:
        routed = _i32(routed).reshape(-1, self.K)
        b = routed.shape[0]
        pred = np.empty((b, self.max_pred), dtype=np.int32)
        n_pred = np.empty(b, dtype=np.int32)
        q_ids = np.empty(self.E, dtype=np.int32)
        q_sc = np.empty(self.E, dtype=np.int32)
        nq = np.zeros(1, dtype=np.int32)
        rc = lib().orc_pred_step(self._h, layer, b, _p(routed), _p(pred), _p(n_pred), _p(q_ids),
                                 _p(q_sc), _p(nq))
        if rc != 0:
            raise AssertionError(f"orc_pred_step failed ({rc})")
        n = int(nq[0])
        return dict(pred_ids=pred, n_pred=n_pred, queue_ids=q_ids[:n].copy(),
                    queue_score=q_sc[:n].copy())

    def stats(self) -> dict:
        o = np.zeros(4, dtype=np.int64)
        lib().orc_pred_stats(self._h, _p(o))
        return dict(steps=int(o[0]), routed=int(o[1]), predicted=int(o[2]), hits=int(o[3]))

    def export(self) -> bytes:
        n = lib().orc_pred_state_bytes(self._h)
        buf = np.empty(n, dtype=np.uint8)
        m = lib().orc_pred_export(self._h, _p(buf))
        assert m == n
        return buf.tobytes()

    def tables(self) -> dict:
        """Decode the canonical state image into arrays."""
        return parse_state(self.export())


def parse_state(blob: bytes) -> dict:
    hdr = np.frombuffer(blob, dtype=np.int32, count=8)
    magic, ver, L, E, K, B, P, built = (int(v) for v in hdr)
    assert magic == 0x53544D50 and ver == 1
    t = int(np.frombuffer(blob, dtype=np.int64, count=1, offset=32)[0])
    pairs = max(L - 1, 0)
    o = 40
    Co = np.frombuffer(blob, dtype=np.uint32, count=pairs * E * E, offset=o).reshape(pairs, E, E)
    o += pairs * E * E * 4
    cid = np.frombuffer(blob, dtype=np.uint8, count=pairs * E * K, offset=o).reshape(pairs, E, K)
    o += pairs * E * K
    cconf = np.frombuffer(blob, dtype=np.uint8, count=pairs * E * K, offset=o).reshape(pairs, E, K)
    o += pairs * E * K
    HT = np.frombuffer(blob, dtype=np.int16, count=B * L * K, offset=o).reshape(B, L, K)
    return dict(L=L, E=E, K=K, B=B, P=P, built=built, t=t, Co=Co, cct_id=cid, cct_conf=cconf,
                HT=HT)


class CacheModel:
    """Integer model of verification, miss loading and prefetch.  window: bits of use history per
    key that rank the victims before recency (0: none); by_turn: among equally used keys evict
    the one whose layer's next turn is furthest; floor: most uses in its window a prefetch
    victim may have (-1: no such test).  window 0 without by_turn is plain LRU."""

    def __init__(self, slots: int, L: int, E: int, window: int = 0, floor: int = -1, by_turn: bool = False):
        self.S, self.L, self.E = slots, L, E
        self._h = lib().orc_cache_create2(slots, L, E, window, floor, int(by_turn))
        if not self._h:
            raise ValueError("bad cache policy")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_cache_destroy(self._h)
            self._h = None

    def step(self, layer, U, next_layer, Q, limit=0) -> dict:
        U, Q = _i32(U), _i32(Q)
        u_slot = np.empty(U.size, dtype=np.int32)
        u_loaded = np.empty(U.size, dtype=np.uint8)
        q_slot = np.empty(max(Q.size, 1), dtype=np.int32)
        rc = lib().orc_cache_step(self._h, layer, _p(U), U.size, next_layer, _p(Q), Q.size, limit,
                                  _p(u_slot), _p(u_loaded), _p(q_slot))
        if rc != 0:
            raise AssertionError("routed experts do not fit in the cache")
        return dict(u_slot=u_slot, u_loaded=u_loaded, q_slot=q_slot[:Q.size])

    def stats(self) -> dict:
        o = np.zeros(7, dtype=np.int64)
        lib().orc_cache_stats(self._h, _p(o))
        names = ["hits", "misses", "pf_issued", "pf_useful", "pf_wasted", "pf_dropped",
                 "pf_resident"]
        return {k: int(v) for k, v in zip(names, o)}

    def tags(self) -> np.ndarray:
        t = np.empty(self.S, dtype=np.int32)
        lib().orc_cache_tags(self._h, _p(t))
        return t


def set_threads(n: int) -> None:
    lib().orc_set_threads(n)


def get_threads() -> int:
    return lib().orc_get_threads()
