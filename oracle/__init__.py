"""ctypes front end of the CPU oracle (``moe_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg may
import this; the CUDA package never does.  Every function takes and returns host numpy arrays.
bf16 tensors are ``uint16`` arrays of bit patterns; ``dtype`` is 0 for fp32, 1 for bf16.

The steps are those of Section II-A of the paper (routing, dispatch, expert computation,
combine, scaling); the dispatch layout is the dense per-expert packing of Section IV-B.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_SO = os.path.join(_HERE, "libmoe_oracle.so")
_lib = None

FP32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved). Returns the path of the shared object."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               _SRC, "-o", _SO, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _storage(a: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == FP32 else np.uint16
    assert a.dtype == want, f"expected {want}, got {a.dtype}"
    return np.ascontiguousarray(a)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def logits(x, wr, bias, dtype):
    T, H = x.shape
    E = wr.shape[0]
    x, wr = _storage(x, dtype), _storage(wr, dtype)
    b = None if bias is None else np.ascontiguousarray(bias, np.float32)
    out = np.empty((T, E), np.float32)
    _check(lib().oracle_logits(T, H, E, dtype, _p(x), _p(wr), _p(b), _p(out)), "oracle_logits")
    return out


def topk(lg, K, renormalize=0):
    lg = np.ascontiguousarray(lg, np.float32)
    T, E = lg.shape
    idx = np.empty((T, K), np.int32)
    w = np.empty((T, K), np.float32)
    _check(lib().oracle_topk(T, E, K, int(renormalize), _p(lg), _p(idx), _p(w)), "oracle_topk")
    return idx, w


def route(x, wr, bias, K, dtype, renormalize=0):
    """Returns (topk_idx[T,K] int32, topk_w[T,K] fp32, logits[T,E] fp32)."""
    T, H = x.shape
    E = wr.shape[0]
    x, wr = _storage(x, dtype), _storage(wr, dtype)
    b = None if bias is None else np.ascontiguousarray(bias, np.float32)
    idx = np.empty((T, K), np.int32)
    w = np.empty((T, K), np.float32)
    lg = np.empty((T, E), np.float32)
    _check(lib().oracle_route(T, H, E, K, dtype, int(renormalize), _p(x), _p(wr), _p(b), _p(idx), _p(w),
                              _p(lg)), "oracle_route")
    return idx, w, lg


def dispatch(x, topk_idx, E, R, dtype, want_rows=True):
    """Returns dict(count[E], offset[E+1], rank_count[R], recv[T*K,H] or None, src[T*K], slot_of[T,K])."""
    T, H = x.shape
    K = topk_idx.shape[1]
    x = _storage(x, dtype)
    idx = np.ascontiguousarray(topk_idx, np.int32)
    count = np.empty(E, np.int32)
    offset = np.empty(E + 1, np.int32)
    rank_count = np.empty(R, np.int32)
    recv = np.empty((T * K, H), x.dtype) if want_rows else None
    src = np.empty(T * K, np.int32)
    slot_of = np.empty((T, K), np.int32)
    _check(lib().oracle_dispatch(T, H, E, R, K, dtype, _p(x), _p(idx), _p(count), _p(offset), _p(rank_count),
                                 _p(recv), _p(src), _p(slot_of)), "oracle_dispatch")
    return dict(count=count, offset=offset, rank_count=rank_count, recv=recv, src=src, slot_of=slot_of)


def round_bf16(a):
    """Nearest bf16 value (ties to even) of every element of an fp64 array, as fp64."""
    a = np.ascontiguousarray(a, np.float64)
    f = lib().oracle_round_bf16
    f.restype, f.argtypes = ctypes.c_double, [ctypes.c_double]
    return np.array([f(float(v)) for v in a.ravel()], np.float64).reshape(a.shape)


def expert_ffn(recv, offset, wg, wu, wd, dtype, bf16_storage=False):
    """wg/wu/wd: sequences of E per-expert arrays ([F,H],[F,H],[H,F]); None allowed for empty experts.
    bf16_storage: the diagnostic restatement that rounds the SwiGLU intermediate and the output rows to
    bf16 (what the CUDA path stores), sums still in fp64.

    Returns out[rows,H] fp64."""
    rows, H = recv.shape
    E = len(wg)
    recv = _storage(recv, dtype)
    offset = np.ascontiguousarray(offset, np.int32)
    F = next(a.shape[0] for a in wg if a is not None)
    keep = []

    def ptrs(ws):
        arr = (ctypes.c_void_p * E)()
        for e, a in enumerate(ws):
            if a is None:
                arr[e] = None
            else:
                a = _storage(a, dtype)
                keep.append(a)
                arr[e] = a.ctypes.data
        return arr

    out = np.empty((rows, H), np.float64)
    fn = lib().oracle_expert_ffn_stored if bf16_storage else lib().oracle_expert_ffn
    _check(fn(H, F, E, dtype, _p(recv), _p(offset), ptrs(wg), ptrs(wu), ptrs(wd), _p(out)), "oracle_expert_ffn")
    return out


def identity_ffn(recv, dtype):
    rows, H = recv.shape
    recv = _storage(recv, dtype)
    out = np.empty((rows, H), np.float64)
    lib().oracle_identity_ffn.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                          ctypes.c_void_p]
    _check(lib().oracle_identity_ffn(rows, H, dtype, _p(recv), _p(out)), "oracle_identity_ffn")
    return out


def combine(rows, slot_of, topk_w, bf16_storage=False):
    """bf16_storage: the diagnostic restatement that rounds y to bf16."""
    rows = np.ascontiguousarray(rows, np.float64)
    T, K = slot_of.shape
    H = rows.shape[1]
    slot_of = np.ascontiguousarray(slot_of, np.int32)
    topk_w = np.ascontiguousarray(topk_w, np.float32)
    y = np.empty((T, H), np.float64)
    fn = lib().oracle_combine_stored if bf16_storage else lib().oracle_combine
    _check(fn(T, H, K, _p(rows), _p(slot_of), _p(topk_w), _p(y)), "oracle_combine")
    return y


def tp_expand(idx, w, wg, wu, wd, S):
    """Expert + tensor parallelism as Section VII of the paper puts it: every TP shard of an expert has a receive
    region of its own and every row is stored to all of them.  Shard s of expert e holds rows [s*F/S, (s+1)*F/S)
    of the gate and up matrices and the matching columns of the down matrix; it is listed as expert e*S + s.
    Returns the routing result with every pick listed once per shard (same weight) and the sliced weights."""
    T, K = idx.shape
    idx_e = (idx[:, :, None].astype(np.int64) * S + np.arange(S)[None, None, :]).reshape(T, K * S).astype(np.int32)
    w_e = np.repeat(w, S, axis=1)
    if wg is None:
        return idx_e, w_e, None, None, None
    wg_e, wu_e, wd_e = [], [], []
    for e in range(len(wg)):
        for s in range(S):
            if wg[e] is None:
                wg_e.append(None), wu_e.append(None), wd_e.append(None)
                continue
            Fs = wg[e].shape[0] // S
            wg_e.append(np.ascontiguousarray(wg[e][s * Fs:(s + 1) * Fs, :]))
            wu_e.append(np.ascontiguousarray(wu[e][s * Fs:(s + 1) * Fs, :]))
            wd_e.append(np.ascontiguousarray(wd[e][:, s * Fs:(s + 1) * Fs]))
    return idx_e, w_e, wg_e, wu_e, wd_e


def layer(x, wr, bias, wg, wu, wd, E, R, K, dtype, renormalize=0, identity_experts=False, bf16_storage=False,
          tp_shards=1):
    """The whole layer: route -> dispatch -> experts -> combine. Returns dict with every stage's output.
    bf16_storage: the diagnostic restatement (intermediate, expert rows and y rounded to bf16).
    tp_shards = S > 1: every expert is cut into S TP shards (see tp_expand); topk_idx, topk_w, slot_of and the
    dispatch outputs are then those of the E*S shards, and y adds the shards' partial rows."""
    idx, w, lg = route(x, wr, bias, K, dtype, renormalize)
    if tp_shards > 1:
        idx, w, wg, wu, wd = tp_expand(idx, w, wg, wu, wd, tp_shards)
        E = E * tp_shards
    d = dispatch(x, idx, E, R, dtype)
    if identity_experts:
        rows = identity_ffn(d["recv"], dtype)
    else:
        rows = expert_ffn(d["recv"], d["offset"], wg, wu, wd, dtype, bf16_storage=bf16_storage)
    y = combine(rows, d["slot_of"], w, bf16_storage=bf16_storage)
    return dict(topk_idx=idx, topk_w=w, logits=lg, out_rows=rows, y=y, **d)
