"""Python face of the CPU oracle -- TEST INFRASTRUCTURE, not product code.

Wraps `spd_oracle.c` (float64, OpenMP over (user, query head)) with ctypes and adds a
NumPy brute-force routine for tiny dense inputs.  Nothing here imports or calls the CUDA
library.  Arrays are NumPy; bf16 data is passed as its uint16 bit pattern.

Functions (each follows the passage named in spd_oracle.c):
  full(...)        unpartitioned softmax(scale q K^T) V            (Eq. 1, left side)
  partial(...)     (O, m, l) of one partition or token range       (Sec. 4.2)
  merge_n(...)     n-way log-sum-exp merge, optional normalise     (Theorem 1, repeated)
  merge_alpha(...) two-way merge with the printed coefficients     (Sec. 4.2)
  brute_force(...) dense triple loop, no max subtraction           (Sec. 2.1 definition)
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spd_oracle.c")
_LIB = os.path.join(_HERE, "libspd_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle's C file with gcc (idempotent)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _KV(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("num_pages", C.c_int64),
                ("page_indptr", C.c_void_p), ("page_indices", C.c_void_p), ("seq_lens", C.c_void_p)]


class _Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("page_size", C.c_int32), ("dtype", C.c_int32),
                ("sm_scale", C.c_double)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.spd_oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(_load().spd_oracle_num_threads())


@dataclass
class KV:
    """One partition as NumPy arrays; pools are float32 or uint16 (bf16 bits), [pages, Hkv, P, D]."""
    k_pool: np.ndarray
    v_pool: np.ndarray
    page_indptr: np.ndarray
    page_indices: np.ndarray
    seq_lens: np.ndarray

    def __post_init__(self):
        self.k_pool = np.ascontiguousarray(self.k_pool)
        self.v_pool = np.ascontiguousarray(self.v_pool)
        self.page_indptr = np.ascontiguousarray(self.page_indptr, dtype=np.int32)
        self.page_indices = np.ascontiguousarray(self.page_indices, dtype=np.int32)
        self.seq_lens = np.ascontiguousarray(self.seq_lens, dtype=np.int32)

    def c(self) -> _KV:
        return _KV(self.k_pool.ctypes.data, self.v_pool.ctypes.data, self.k_pool.shape[0],
                   self.page_indptr.ctypes.data, self.page_indices.ctypes.data, self.seq_lens.ctypes.data)


def _shape(q: np.ndarray, kv: KV, sm_scale: float) -> _Shape:
    B, Hq, D = q.shape
    _, Hkv, P, D2 = kv.k_pool.shape
    assert D == D2 and Hq % Hkv == 0
    if q.dtype == np.float32:
        dt = F32
    elif q.dtype == np.uint16:
        dt = BF16
    else:
        raise TypeError("q must be float32 or uint16 (bf16 bits)")
    assert kv.k_pool.dtype == q.dtype and kv.v_pool.dtype == q.dtype
    return _Shape(B, Hq, Hkv, D, P, dt, float(sm_scale))


def full(q: np.ndarray, priv: Optional[KV], pub: Optional[KV], sm_scale: float,
         users: Optional[Tuple[int, int]] = None) -> np.ndarray:
    """Unpartitioned attention over private-then-public tokens; returns [B, Hq, D] float64."""
    lib = _load()
    q = np.ascontiguousarray(q)
    ref = priv if priv is not None else pub
    sh = _shape(q, ref, sm_scale)
    y = np.zeros(q.shape, dtype=np.float64)
    lo, hi = users if users is not None else (0, q.shape[0])
    cp = priv.c() if priv is not None else None
    cq = pub.c() if pub is not None else None
    lib.spd_oracle_full(C.byref(sh), C.c_void_p(q.ctypes.data),
                        C.byref(cp) if cp is not None else None,
                        C.byref(cq) if cq is not None else None,
                        C.c_int(lo), C.c_int(hi), C.c_void_p(y.ctypes.data))
    return y


def partial(q: np.ndarray, kv: KV, sm_scale: float, tok_lo: int = 0, tok_hi: int = 2 ** 62):
    """(O [B,Hq,D], m [B,Hq], l [B,Hq]) float64 over tokens [tok_lo, min(tok_hi, len))."""
    lib = _load()
    q = np.ascontiguousarray(q)
    sh = _shape(q, kv, sm_scale)
    B, Hq, D = q.shape
    o = np.zeros((B, Hq, D), dtype=np.float64)
    m = np.zeros((B, Hq), dtype=np.float64)
    l = np.zeros((B, Hq), dtype=np.float64)
    ckv = kv.c()
    lib.spd_oracle_partial(C.byref(sh), C.c_void_p(q.ctypes.data), C.byref(ckv),
                           C.c_int64(tok_lo), C.c_int64(tok_hi),
                           C.c_void_p(o.ctypes.data), C.c_void_p(m.ctypes.data), C.c_void_p(l.ctypes.data))
    return o, m, l


def merge_n(parts_o, parts_m, parts_l, normalise: bool = True):
    """Merge n partials ([n,...,D], [n,...], [n,...]); returns (O, m, l, Y or None)."""
    lib = _load()
    po = np.ascontiguousarray(parts_o, dtype=np.float64)
    pm = np.ascontiguousarray(parts_m, dtype=np.float64)
    pl = np.ascontiguousarray(parts_l, dtype=np.float64)
    n, D = po.shape[0], po.shape[-1]
    rows = int(np.prod(pm.shape[1:]))
    o = np.zeros(po.shape[1:], dtype=np.float64)
    m = np.zeros(pm.shape[1:], dtype=np.float64)
    l = np.zeros(pm.shape[1:], dtype=np.float64)
    y = np.zeros(po.shape[1:], dtype=np.float64) if normalise else None
    lib.spd_oracle_merge_n(C.c_int(n), C.c_int64(rows), C.c_int(D), C.c_void_p(po.ctypes.data),
                           C.c_void_p(pm.ctypes.data), C.c_void_p(pl.ctypes.data),
                           C.c_void_p(o.ctypes.data), C.c_void_p(m.ctypes.data), C.c_void_p(l.ctypes.data),
                           C.c_void_p(y.ctypes.data) if y is not None else None)
    return o, m, l, y


def merge_alpha(o_in, m_in, l_in, o_out, m_out, l_out) -> np.ndarray:
    """Two-way merge with the alpha coefficients; both partitions non-empty."""
    lib = _load()
    arrs = [np.ascontiguousarray(a, dtype=np.float64) for a in (o_in, m_in, l_in, o_out, m_out, l_out)]
    D = arrs[0].shape[-1]
    rows = int(np.prod(arrs[1].shape))
    y = np.zeros(arrs[0].shape, dtype=np.float64)
    lib.spd_oracle_merge_alpha(C.c_int64(rows), C.c_int(D), *[C.c_void_p(a.ctypes.data) for a in arrs],
                               C.c_void_p(y.ctypes.data))
    return y


def partitioned(q: np.ndarray, priv: KV, pub: KV, sm_scale: float) -> np.ndarray:
    """Private partial, public partial, merge: the decode step as the method splits it."""
    oi, mi, li = partial(q, priv, sm_scale)
    oo, mo, lo = partial(q, pub, sm_scale)
    return merge_n(np.stack([oi, oo]), np.stack([mi, mo]), np.stack([li, lo]))[3]


def brute_force(q: np.ndarray, k: np.ndarray, v: np.ndarray, sm_scale: float) -> np.ndarray:
    """softmax(scale q k^T) v for ONE query vector over dense [n, D] keys/values.

    Pure-Python triple loop straight from the definition: exp of the raw score, no maximum
    subtracted, denominators summed term by term.  Only for tiny inputs with small scores.
    """
    n, D = k.shape
    y = [0.0] * D
    den = 0.0
    e = []
    for i in range(n):
        s = 0.0
        for d in range(D):
            s += float(q[d]) * float(k[i, d])
        e.append(float(np.exp(sm_scale * s)))
        den += e[-1]
    for i in range(n):
        for d in range(D):
            y[d] += e[i] / den * float(v[i, d])
    return np.asarray(y, dtype=np.float64)


def bf16_bits(x) -> np.ndarray:
    """Reinterpret a torch bf16 tensor (CPU) as a uint16 NumPy array (no arithmetic)."""
    import torch
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def kv_from_torch(part) -> KV:
    """Adapter from the workload generator's PagedKV (CPU tensors) to the oracle's KV."""
    import torch

    def arr(t):
        return bf16_bits(t) if t.dtype == torch.bfloat16 else t.contiguous().numpy()
    return KV(arr(part.k_pool), arr(part.v_pool), part.page_indptr.numpy(), part.page_indices.numpy(),
              part.seq_lens.numpy())


def q_from_torch(q) -> np.ndarray:
    import torch
    return bf16_bits(q) if q.dtype == torch.bfloat16 else q.contiguous().numpy()


def append(kv: KV, k_new: np.ndarray, v_new: np.ndarray) -> np.ndarray:
    """Append one token per user to a partition, in place (protocol step 3a; Fig. 3 step 2).

    k_new, v_new: [B, Hkv, D] in the pools' dtype.  The row of user u goes to token position
    len_u, i.e. page page_indices[page_indptr[u] + len_u // P], slot len_u % P, and len_u grows by
    one.  A user whose listed pages are full is left untouched.  Returns a bool array: appended or not.
    Pure indexing, written out as loops.
    """
    B, Hkv, D = k_new.shape
    P = kv.k_pool.shape[2]
    done = np.zeros(B, dtype=bool)
    for u in range(B):
        t = int(kv.seq_lens[u])
        cap = int(kv.page_indptr[u + 1]) - int(kv.page_indptr[u])
        if t < 0 or t >= cap * P:
            continue
        page = int(kv.page_indices[int(kv.page_indptr[u]) + t // P])
        for h in range(Hkv):
            for d in range(D):
                kv.k_pool[page, h, t % P, d] = k_new[u, h, d]
                kv.v_pool[page, h, t % P, d] = v_new[u, h, d]
        kv.seq_lens[u] = t + 1
        done[u] = True
    return done


def watched_mass(q: np.ndarray, priv: KV, pub: Optional[KV], sm_scale: float, tok_lo, tok_hi):
    """Share of the softmax mass that sits on tokens [tok_lo[u], tok_hi[u]) of the private partition
    (Sec. 2.4.4 / 7.1.1: attention paid to the watched instruction).

    Returns (share_full [B, Hq], share_private [B, Hq]): relative to the attention over both partitions
    and over the private partition alone.  Written from the definition: with the partials
    (m_w, l_w) of the watched range, (m_in, l_in) of the private and (m_out, l_out) of the public
    partition, the mass of a set is l * exp(m) and a share is a ratio of masses.
    """
    B, Hq, _ = q.shape
    _, m_in, l_in = partial(q, priv, sm_scale)
    if pub is not None:
        _, m_out, l_out = partial(q, pub, sm_scale)
    else:
        m_out, l_out = np.full((B, Hq), -np.inf), np.zeros((B, Hq))
    full = np.zeros((B, Hq))
    own = np.zeros((B, Hq))
    for u in range(B):
        lo, hi = max(int(tok_lo[u]), 0), int(tok_hi[u])
        if hi <= lo:
            continue
        _, m_w, l_w = partial(q, priv, sm_scale, lo, hi)
        for h in range(Hq):
            if l_w[u, h] == 0.0:
                continue
            M = max(m_in[u, h], m_out[u, h])
            mass_w = l_w[u, h] * np.exp(m_w[u, h] - M)
            mass_in = l_in[u, h] * np.exp(m_in[u, h] - M)
            mass_out = l_out[u, h] * np.exp(m_out[u, h] - M) if l_out[u, h] > 0 else 0.0
            full[u, h] = mass_w / (mass_in + mass_out)
            own[u, h] = mass_w / mass_in
    return full, own


def prefill(q: np.ndarray, k: np.ndarray, v: np.ndarray, tok_indptr, sm_scale: float, rows=None) -> np.ndarray:
    """Causal self-attention over each user's prompt (protocol step 2).

    q [T, Hq, D], k, v [T, Hkv, D] (float32 or uint16 bf16 bits), users laid end to end with token offsets
    tok_indptr [B+1].  Returns y [len(rows), Hq, D] float64 for the listed global token indices
    (all tokens when rows is None)."""
    lib = _load()
    q, k, v = (np.ascontiguousarray(a) for a in (q, k, v))
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    ip = np.ascontiguousarray(tok_indptr, dtype=np.int32)
    rows = np.arange(T, dtype=np.int64) if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    dt = F32 if q.dtype == np.float32 else BF16
    sh = _Shape(len(ip) - 1, Hq, Hkv, D, 16, dt, float(sm_scale))
    y = np.zeros((len(rows), Hq, D), dtype=np.float64)
    lib.spd_oracle_prefill(C.byref(sh), C.c_void_p(q.ctypes.data), C.c_void_p(k.ctypes.data), C.c_void_p(v.ctypes.data),
                           C.c_void_p(ip.ctypes.data), C.c_void_p(rows.ctypes.data), C.c_int64(len(rows)),
                           C.c_void_p(y.ctypes.data))
    return y


def write_prompt_kv(kv: KV, k: np.ndarray, v: np.ndarray, tok_indptr) -> None:
    """Store every prompt token's K and V row in the paged cache, in place, and set seq_lens (what prefill
    leaves behind for decode).  Token t of user u goes to page page_indices[page_indptr[u] + t // P], slot
    t % P.  Pure indexing."""
    P = kv.k_pool.shape[2]
    for u in range(len(tok_indptr) - 1):
        a, b = int(tok_indptr[u]), int(tok_indptr[u + 1])
        for t in range(b - a):
            page = int(kv.page_indices[int(kv.page_indptr[u]) + t // P])
            kv.k_pool[page, :, t % P, :] = k[a + t]
            kv.v_pool[page, :, t % P, :] = v[a + t]
        kv.seq_lens[u] = b - a
