"""Test-side input plumbing: packs dense per-user K/V into the paged layout (indexing only)."""
import numpy as np

from oracle import spd_oracle as orc


def dense_to_paged(ks, vs, page_size=16, rng=None, extra_pages=3, dtype=np.float32):
    """ks[u], vs[u]: arrays [Hkv, L_u, D] (L_u may be 0).  Returns an oracle KV whose pages are
    handed out in a shuffled order; every unoccupied slot is NaN."""
    rng = rng or np.random.default_rng(0)
    B = len(ks)
    Hkv, _, D = ks[0].shape
    lens = np.array([k.shape[1] for k in ks], dtype=np.int64)
    need = (lens + page_size - 1) // page_size
    indptr = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(need, out=indptr[1:])
    total = int(indptr[-1])
    num_pages = total + extra_pages
    perm = rng.permutation(num_pages)
    indices = perm[:total].astype(np.int32)
    kp = np.full((num_pages, Hkv, page_size, D), np.nan, dtype=np.float32)
    vp = np.full((num_pages, Hkv, page_size, D), np.nan, dtype=np.float32)
    for u in range(B):
        for t in range(int(lens[u])):
            pg = indices[indptr[u] + t // page_size]
            kp[pg, :, t % page_size, :] = ks[u][:, t, :]
            vp[pg, :, t % page_size, :] = vs[u][:, t, :]
    if dtype == np.uint16:
        kp, vp = f32_to_bf16_bits(kp), f32_to_bf16_bits(vp)
    return orc.KV(kp, vp, indptr.astype(np.int32), indices, lens.astype(np.int32))


def f32_to_bf16_bits(x):
    """Truncate float32 values that are already bf16-representable to their 16-bit pattern."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (bits >> 16).astype(np.uint16)


def round_to_bf16(x):
    """Round float32 to the nearest bf16-representable float32 (ties to even), NaN kept."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).float().numpy()
