"""Pins for the CPU oracle: things the paper and the mathematics fix, none of them the oracle itself.

Each test is built so that one plausible mistake in oracle/spd_oracle.c (a dropped term, a wrong
sign, a transposed index, a wrong head map, a mis-decoded bf16, a mis-indexed page) fails it.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import workloads as wl
from tests.helpers import dense_to_paged, f32_to_bf16_bits, round_to_bf16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_dense(rng, lens, Hkv, D, scale=1.0):
    ks = [rng.standard_normal((Hkv, L, D)).astype(np.float32) * scale for L in lens]
    vs = [rng.standard_normal((Hkv, L, D)).astype(np.float32) for L in lens]
    return ks, vs


# ---------------------------------------------------------------- hand-derived golden (Thm 1, Sec. 4.2)
def _parse_golden(path):
    consts = {"LN2": math.log(2), "LN3": math.log(3), "LN4": math.log(4)}
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        rows = [[consts.get(tok, None) if tok in consts else float(tok) for tok in r.split()]
                for r in rest.split("|")]
        out[key] = np.array(rows, dtype=np.float64)
    return out


def test_golden_hand_example():
    g = _parse_golden(os.path.join(GOLDEN, "thm1_hand_example.txt"))
    q = g["q"].astype(np.float32).reshape(1, 1, 2)
    kin = dense_to_paged([g["k_in"].astype(np.float32)[None]], [g["v_in"].astype(np.float32)[None]])
    kout = dense_to_paged([g["k_out"].astype(np.float32)[None]], [g["v_out"].astype(np.float32)[None]])
    tol = 1e-6  # ln(i) is rounded to float32 on input
    y = orc.full(q, kin, kout, 1.0)
    assert np.allclose(y[0, 0], g["y"][0], atol=tol)
    oi, mi, li = orc.partial(q, kin, 1.0)
    oo, mo, lo = orc.partial(q, kout, 1.0)
    assert abs(mi[0, 0] - g["m_in"][0, 0]) < tol and abs(li[0, 0] - g["l_in"][0, 0]) < tol
    assert abs(mo[0, 0] - g["m_out"][0, 0]) < tol and abs(lo[0, 0] - g["l_out"][0, 0]) < tol
    assert np.allclose(oi[0, 0], g["o_in"][0], atol=1e-5) and np.allclose(oo[0, 0], g["o_out"][0], atol=tol)
    ym = orc.merge_n(np.stack([oi, oo]), np.stack([mi, mo]), np.stack([li, lo]))[3]
    assert np.allclose(ym[0, 0], g["y"][0], atol=tol)
    ya = orc.merge_alpha(oi, mi, li, oo, mo, lo)
    assert np.allclose(ya[0, 0], g["y"][0], atol=tol)
    # the printed coefficients: gamma_in/(gamma_in + alpha gamma_out), gamma_out/(gamma_in/alpha + gamma_out)
    alpha = math.exp(mo[0, 0] - mi[0, 0])
    assert abs(li[0, 0] / (li[0, 0] + alpha * lo[0, 0]) - g["coef_in"][0, 0]) < tol
    assert abs(lo[0, 0] / (li[0, 0] / alpha + lo[0, 0]) - g["coef_out"][0, 0]) < tol


# ---------------------------------------------------------------- brute force on tiny inputs
@pytest.mark.parametrize("Hq,Hkv,D", [(2, 2, 4), (4, 2, 8), (4, 1, 4), (8, 8, 64)])
def test_brute_force_tiny(Hq, Hkv, D):
    rng = np.random.default_rng(11 + Hq + D)
    lens_in, lens_out = [37, 1, 16], [5, 40, 0]
    ks, vs = _rand_dense(rng, lens_in, Hkv, D, 0.5)
    ko, vo = _rand_dense(rng, lens_out, Hkv, D, 0.5)
    q = (rng.standard_normal((3, Hq, D)) * 0.5).astype(np.float32)
    kin, kout = dense_to_paged(ks, vs, rng=rng), dense_to_paged(ko, vo, rng=rng)
    scale = 1.0 / math.sqrt(D)
    y_full = orc.full(q, kin, kout, scale)
    y_part = orc.partitioned(q, kin, kout, scale)
    g = Hq // Hkv
    for u in range(3):
        for h in range(Hq):
            kd = np.concatenate([ks[u][h // g], ko[u][h // g]], axis=0)
            vd = np.concatenate([vs[u][h // g], vo[u][h // g]], axis=0)
            yb = orc.brute_force(q[u, h], kd, vd, scale)
            assert np.max(np.abs(y_full[u, h] - yb)) < 1e-12
            assert np.max(np.abs(y_part[u, h] - yb)) < 1e-12


# ---------------------------------------------------------------- Theorem 1: every split point
def test_split_point_identity_every_split():
    rng = np.random.default_rng(5)
    L, Hkv, Hq, D = 45, 2, 4, 8
    ks, vs = _rand_dense(rng, [L, L - 7], Hkv, D)
    q = rng.standard_normal((2, Hq, D)).astype(np.float32)
    kv = dense_to_paged(ks, vs, rng=rng)
    y_full = orc.full(q, kv, None, 0.3)
    for s in range(0, L + 1):
        a = orc.partial(q, kv, 0.3, 0, s)
        b = orc.partial(q, kv, 0.3, s, L)
        y = orc.merge_n(np.stack([a[0], b[0]]), np.stack([a[1], b[1]]), np.stack([a[2], b[2]]))[3]
        assert np.max(np.abs(y - y_full)) < 1e-12, s
    # empty partitions are the identity of the merge and carry (0, -inf, 0)
    e = orc.partial(q, kv, 0.3, L, L)
    assert np.all(e[0] == 0) and np.all(np.isneginf(e[1])) and np.all(e[2] == 0)


def test_nway_and_nested_merge():
    rng = np.random.default_rng(6)
    L, D = 64, 8
    ks, vs = _rand_dense(rng, [L], 1, D, 3.0)   # large scores: stabilisation matters
    q = rng.standard_normal((1, 2, D)).astype(np.float32)
    kv = dense_to_paged(ks, vs, rng=rng)
    y_full = orc.full(q, kv, None, 1.0)
    cuts = [0, 1, 16, 17, 40, 64]
    parts = [orc.partial(q, kv, 1.0, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    O, m, l, y = orc.merge_n(np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]),
                             np.stack([p[2] for p in parts]))
    assert np.max(np.abs(y - y_full)) < 1e-12
    # nested: merge the first three, then that with the rest
    O1, m1, l1, _ = orc.merge_n(np.stack([p[0] for p in parts[:3]]), np.stack([p[1] for p in parts[:3]]),
                                np.stack([p[2] for p in parts[:3]]), normalise=False)
    rest = parts[3:]
    y2 = orc.merge_n(np.stack([O1] + [p[0] for p in rest]), np.stack([m1] + [p[1] for p in rest]),
                     np.stack([l1] + [p[2] for p in rest]))[3]
    assert np.max(np.abs(y2 - y_full)) < 1e-12
    # the merged partial equals the partial computed in one go (gauge-free comparison)
    Of, mf, lf = orc.partial(q, kv, 1.0)
    assert np.allclose(O / l[..., None], Of / lf[..., None], atol=1e-12)
    assert np.allclose(m + np.log(l), mf + np.log(lf), atol=1e-12)
    assert np.allclose(m, mf, atol=0)


def test_alpha_form_matches_max_form():
    rng = np.random.default_rng(7)
    ks, vs = _rand_dense(rng, [33, 8], 2, 16, 2.0)
    ko, vo = _rand_dense(rng, [9, 70], 2, 16, 2.0)
    q = rng.standard_normal((2, 4, 16)).astype(np.float32)
    kin, kout = dense_to_paged(ks, vs, rng=rng), dense_to_paged(ko, vo, rng=rng)
    a, b = orc.partial(q, kin, 0.5), orc.partial(q, kout, 0.5)
    y1 = orc.merge_n(np.stack([a[0], b[0]]), np.stack([a[1], b[1]]), np.stack([a[2], b[2]]))[3]
    y2 = orc.merge_alpha(*a, *b)
    assert np.max(np.abs(y1 - y2)) < 1e-12
    assert np.max(np.abs(y1 - orc.full(q, kin, kout, 0.5))) < 1e-12


# ---------------------------------------------------------------- closed forms
def test_uniform_scores_give_mean_of_v():
    rng = np.random.default_rng(8)
    ks, vs = _rand_dense(rng, [23], 2, 8)
    ko, vo = _rand_dense(rng, [10], 2, 8)
    kin, kout = dense_to_paged(ks, vs, rng=rng), dense_to_paged(ko, vo, rng=rng)
    q = np.zeros((1, 4, 8), dtype=np.float32)  # q = 0: all scores equal
    y = orc.full(q, kin, kout, 1.0)
    for h in range(4):
        mean = np.concatenate([vs[0][h // 2], vo[0][h // 2]]).astype(np.float64).mean(axis=0)
        assert np.max(np.abs(y[0, h] - mean)) < 1e-12
    # identical keys, non-zero query: again the mean; l counts the tokens, m is the common score
    k1 = np.tile(rng.standard_normal((2, 1, 8)).astype(np.float32), (1, 23, 1))
    kin2 = dense_to_paged([k1], vs, rng=rng)
    q2 = rng.standard_normal((1, 4, 8)).astype(np.float32)
    O, m, l = orc.partial(q2, kin2, 0.7)
    assert np.allclose(l, 23.0, atol=1e-12)
    for h in range(4):
        s = 0.7 * float(np.dot(q2[0, h].astype(np.float64), k1[h // 2, 0].astype(np.float64)))
        assert abs(m[0, h] - s) < 1e-12
        assert np.allclose(O[0, h] / l[0, h], vs[0][h // 2].astype(np.float64).mean(axis=0), atol=1e-12)


def test_single_key_returns_its_value():
    rng = np.random.default_rng(9)
    ks, vs = _rand_dense(rng, [1], 2, 8)
    kin = dense_to_paged(ks, vs, rng=rng)
    empty = dense_to_paged([np.zeros((2, 0, 8), np.float32)], [np.zeros((2, 0, 8), np.float32)], rng=rng)
    q = rng.standard_normal((1, 4, 8)).astype(np.float32)
    O, m, l = orc.partial(q, kin, 0.25)
    y = orc.full(q, kin, empty, 0.25)
    y_swapped = orc.full(q, empty, kin, 0.25)
    for h in range(4):
        assert np.array_equal(y[0, h], vs[0][h // 2, 0].astype(np.float64))
        assert np.array_equal(y_swapped[0, h], y[0, h])
        assert l[0, h] == 1.0
        assert abs(m[0, h] - 0.25 * np.dot(q[0, h].astype(np.float64), ks[0][h // 2, 0].astype(np.float64))) < 1e-14
        assert np.array_equal(O[0, h], y[0, h])
    # both partitions empty: zeros, no NaN
    assert np.all(orc.full(q, empty, empty, 0.25) == 0)
    assert np.all(orc.partitioned(q, empty, empty, 0.25) == 0)


def test_dominant_key_duplicate_tokens_and_score_shift():
    rng = np.random.default_rng(10)
    D = 8
    ks, vs = _rand_dense(rng, [20], 1, D)
    q = rng.standard_normal((1, 1, D)).astype(np.float32)
    # one key aligned with q and scaled up dominates
    ks[0][0, 13] = q[0, 0] * 40.0
    kv = dense_to_paged(ks, vs, rng=rng)
    y = orc.full(q, kv, None, 1.0)
    assert np.max(np.abs(y[0, 0] - vs[0][0, 13])) < 1e-9
    # duplicating every token leaves Y and m unchanged and doubles l
    ks2 = [np.concatenate([ks[0], ks[0]], axis=1)]
    vs2 = [np.concatenate([vs[0], vs[0]], axis=1)]
    kv2 = dense_to_paged(ks2, vs2, rng=rng)
    O1, m1, l1 = orc.partial(q, kv, 0.1)
    O2, m2, l2 = orc.partial(q, kv2, 0.1)
    assert np.allclose(l2, 2 * l1, rtol=1e-14) and np.array_equal(m1, m2)
    assert np.allclose(O2 / l2[..., None], O1 / l1[..., None], atol=1e-13)
    # adding c*e to every key with <q, e> = 1 shifts every score by scale*c: Y same, m moves
    e = (q[0, 0] / np.dot(q[0, 0], q[0, 0])).astype(np.float64)
    c = 2.0
    ks3 = [(ks[0].astype(np.float64) + c * e).astype(np.float32)]
    kv3 = dense_to_paged(ks3, vs, rng=rng)
    O3, m3, l3 = orc.partial(q, kv3, 0.1)
    assert np.allclose(m3 - m1, 0.1 * c, atol=1e-5)
    assert np.allclose(O3 / l3[..., None], O1 / l1[..., None], atol=1e-5)


# ---------------------------------------------------------------- textbook dense softmax
def test_matches_dense_numpy_and_torch_sdpa():
    rng = np.random.default_rng(12)
    B, H, D, L = 2, 4, 16, 50
    ks, vs = _rand_dense(rng, [L] * B, H, D)
    q = rng.standard_normal((B, H, D)).astype(np.float32)
    kv = dense_to_paged(ks, vs, rng=rng)
    scale = 1.0 / math.sqrt(D)
    y = orc.full(q, kv, None, scale)
    K = np.stack(ks).astype(np.float64)   # [B,H,L,D]
    V = np.stack(vs).astype(np.float64)
    S = np.einsum("bhd,bhld->bhl", q.astype(np.float64), K) * scale
    Pm = np.exp(S - S.max(-1, keepdims=True))
    Pm /= Pm.sum(-1, keepdims=True)
    y_np = np.einsum("bhl,bhld->bhd", Pm, V)
    assert np.max(np.abs(y - y_np)) < 1e-12
    y_t = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double()[:, :, None, :], torch.from_numpy(K), torch.from_numpy(V), scale=scale)
    assert np.max(np.abs(y - y_t[:, :, 0, :].numpy())) < 1e-12


# ---------------------------------------------------------------- head map, paging, bf16 decoding
def test_gqa_head_map_is_contiguous_groups():
    Hq, Hkv, D, L = 8, 2, 4, 5
    ks = [np.ones((Hkv, L, D), np.float32)]
    vs = [np.stack([np.full((L, D), 100.0 * (kvh + 1), np.float32) for kvh in range(Hkv)])]
    kv = dense_to_paged(ks, vs)
    q = np.ones((1, Hq, D), np.float32)
    y = orc.full(q, kv, None, 1.0)
    for h in range(Hq):
        assert np.allclose(y[0, h], 100.0 * (h // (Hq // Hkv) + 1))


def test_indexing_probe_one_hot_query():
    """A huge score on exactly one token makes the output that token's V, which encodes
    (user, kv head, token, d) -- so any mis-indexed page, slot or head shows as a wrong integer."""
    rng = np.random.default_rng(13)
    B, Hkv, g, D, P = 3, 2, 2, 8, 16
    lens = [50, 16, 33]
    ks, vs = [], []
    for u, L in enumerate(lens):
        k = np.zeros((Hkv, L, D), np.float32)
        v = np.zeros((Hkv, L, D), np.float32)
        for kvh in range(Hkv):
            for t in range(L):
                v[kvh, t] = [u, kvh, t, 0, 1, 2, 3, 4]
        ks.append(k)
        vs.append(v)
    target = {(u, h): int(rng.integers(0, lens[u])) for u in range(B) for h in range(Hkv * g)}
    # each query head looks along its own axis; exactly one token per (user, kv head, axis) has
    # a large component there
    q = np.zeros((B, Hkv * g, D), np.float32)
    for (u, h), t in target.items():
        q[u, h, h] = 1.0
        ks[u][h // g, t, h] = 200.0
    kv = dense_to_paged(ks, vs, page_size=P, rng=rng)
    y = orc.full(q, kv, None, 1.0)
    for (u, h), t in target.items():
        assert np.array_equal(y[u, h], np.array([u, h // g, t, 0, 1, 2, 3, 4], np.float64)), (u, h, t)


def test_bf16_bits_are_widened_exactly_and_page_shuffle_is_invisible():
    rng = np.random.default_rng(14)
    lens = [19, 40]
    ks, vs = _rand_dense(rng, lens, 2, 8)
    ks = [round_to_bf16(k) for k in ks]
    vs = [round_to_bf16(v) for v in vs]
    q = round_to_bf16(rng.standard_normal((2, 4, 8)).astype(np.float32))
    kv32 = dense_to_paged(ks, vs, rng=np.random.default_rng(1))
    kv16a = dense_to_paged(ks, vs, rng=np.random.default_rng(2), dtype=np.uint16)
    kv16b = dense_to_paged(ks, vs, rng=np.random.default_rng(3), dtype=np.uint16, extra_pages=9)
    y32 = orc.full(q, kv32, None, 0.35)
    y16a = orc.full(f32_to_bf16_bits(q), kv16a, None, 0.35)
    y16b = orc.full(f32_to_bf16_bits(q), kv16b, None, 0.35)
    assert np.array_equal(y32, y16a)      # same values, two encodings
    assert np.array_equal(y16a, y16b)     # physical page order changes nothing, bit for bit


def test_batch_independence_and_user_permutation():
    w = wl.make_workload(dict(batch=5, hq=4, hkv=2, d=16, dtype="f32", lin=("uniform", 1, 70),
                              lout=("uniform", 0, 40), seed=3), slack=True)
    q = orc.q_from_torch(w.q)
    kin, kout = orc.kv_from_torch(w.priv), orc.kv_from_torch(w.pub)
    y = orc.full(q, kin, kout, w.sm_scale)
    assert np.all(np.isfinite(y))         # NaN-poisoned tails, slack and free pages are never read
    assert np.max(np.abs(y - orc.partitioned(q, kin, kout, w.sm_scale))) < 1e-12
    for u in range(w.batch):              # each user alone, through the same pools
        def one(kv):
            lo, hi = int(kv.page_indptr[u]), int(kv.page_indptr[u + 1])
            return orc.KV(kv.k_pool, kv.v_pool, np.array([0, hi - lo]), kv.page_indices[lo:hi],
                          kv.seq_lens[u:u + 1])
        y1 = orc.full(q[u:u + 1], one(kin), one(kout), w.sm_scale)
        assert np.array_equal(y1[0], y[u])


def test_workload_generator_recipes():
    """Lengths follow the stated recipes; pools carry NaN exactly where no token lives."""
    for name, cfg in wl.CONFIGS.items():
        lin, lout = wl.make_lengths(cfg)
        for arr, spec in ((lin, cfg["lin"]), (lout, cfg["lout"])):
            lo, hi = (spec[1], spec[1]) if spec[0] == "const" else (spec[-2], spec[-1])
            assert arr.min() >= lo and arr.max() <= hi and len(arr) == cfg["batch"]
        lin2, _ = wl.make_lengths(cfg)
        assert np.array_equal(lin, lin2)
    w = wl.make_workload("c1_tiny_mha")
    assert w.q.shape == (4, 8, 64) and w.kv_bytes() == 4 * (256 + 32) * 2 * 8 * 64 * 4
    w = wl.make_workload(dict(batch=3, hq=2, hkv=1, d=8, dtype="bf16", lin=("uniform", 1, 40),
                              lout=("const", 0), seed=1), slack=True)
    n_tok = int(w.priv.seq_lens.sum())
    assert int((~torch.isnan(w.priv.k_pool.float()[..., 0])).sum()) == n_tok
    assert w.pub.page_indices.numel() >= 0 and torch.isnan(w.pub.k_pool.float()).all()


# ---------------------------------------------------------------- append of the new token (step 3a)
def test_append_then_attend_equals_dense_concatenation():
    rng = np.random.default_rng(21)
    Hkv, Hq, D, P = 2, 4, 8, 16
    lens = [15, 16, 0, 31]                      # last slot of a page, first slot of a fresh page, empty, mid-page
    ks, vs = _rand_dense(rng, lens, Hkv, D)
    kv = dense_to_paged(ks, vs, rng=rng)
    # give every user one spare page beyond what its tokens need, except user 3 (full after one more token)
    need = [(n + P - 1) // P for n in lens]
    cap = [need[0], need[1] + 1, 1, need[3]]
    indptr = np.concatenate([[0], np.cumsum(cap)]).astype(np.int32)
    spare = iter(sorted(set(range(kv.k_pool.shape[0])) - set(kv.page_indices.tolist())))   # the 3 unused pages
    indices = []
    for u in range(4):
        own = list(kv.page_indices[kv.page_indptr[u]:kv.page_indptr[u + 1]])
        while len(own) < cap[u]:
            own.append(next(spare))
        indices += own
    kv = orc.KV(kv.k_pool, kv.v_pool, indptr, np.array(indices, np.int32), kv.seq_lens)
    before_k = kv.k_pool.copy()
    k_new = rng.standard_normal((4, Hkv, D)).astype(np.float32)
    v_new = rng.standard_normal((4, Hkv, D)).astype(np.float32)
    done = orc.append(kv, k_new, v_new)
    assert done.tolist() == [True, True, True, True] and kv.seq_lens.tolist() == [16, 17, 1, 32]
    # exactly one row per (user, kv head) changed
    changed = ~((before_k == kv.k_pool) | (np.isnan(before_k) & np.isnan(kv.k_pool)))
    assert int(changed.any(axis=-1).sum()) == 4 * Hkv
    q = rng.standard_normal((4, Hq, D)).astype(np.float32)
    y = orc.full(q, kv, None, 0.4)
    for u in range(4):
        for h in range(Hq):
            kd = np.concatenate([ks[u][h // 2], k_new[u, h // 2][None]], axis=0)
            vd = np.concatenate([vs[u][h // 2], v_new[u, h // 2][None]], axis=0)
            assert np.max(np.abs(y[u, h] - orc.brute_force(q[u, h], kd, vd, 0.4))) < 1e-12
    # users 0 and 3 are now full: a second append leaves them alone, the others grow
    snap = (kv.k_pool.copy(), kv.seq_lens.copy())
    done = orc.append(kv, k_new, v_new)
    assert done.tolist() == [False, True, True, False] and kv.seq_lens.tolist() == [16, 18, 2, 32]
    for u in (0, 3):
        pages = kv.page_indices[kv.page_indptr[u]:kv.page_indptr[u + 1]]
        assert np.array_equal(np.nan_to_num(kv.k_pool[pages]), np.nan_to_num(snap[0][pages]))


# ---------------------------------------------------------------- watched attention mass (Sec. 2.4.4)
def test_watched_mass_is_the_sum_of_softmax_probabilities():
    rng = np.random.default_rng(31)
    B, Hkv, Hq, D = 3, 2, 4, 8
    lin, lout = [40, 7, 16], [9, 0, 3]
    ks, vs = _rand_dense(rng, lin, Hkv, D)
    ko, vo = _rand_dense(rng, lout, Hkv, D)
    kin, kout = dense_to_paged(ks, vs, rng=rng), dense_to_paged(ko, vo, rng=rng)
    q = rng.standard_normal((B, Hq, D)).astype(np.float32)
    lo, hi = np.array([5, 0, 16]), np.array([23, 7, 30])     # the last range lies past the partition: watches nothing
    full, own = orc.watched_mass(q, kin, kout, 0.6, lo, hi)
    for u in range(B):
        for h in range(Hq):
            K = np.concatenate([ks[u][h // 2], ko[u][h // 2]]).astype(np.float64)
            s = 0.6 * K @ q[u, h].astype(np.float64)
            pr = np.exp(s - s.max())
            pr /= pr.sum()
            a, b = min(lo[u], lin[u]), min(hi[u], lin[u])
            assert abs(full[u, h] - pr[a:b].sum()) < 1e-12
            pin = np.exp(s[:lin[u]] - s[:lin[u]].max())
            pin /= pin.sum()
            assert abs(own[u, h] - pin[a:b].sum()) < 1e-12
    # the whole private partition with no public tokens holds all the mass; disjoint ranges add up
    f1, o1 = orc.watched_mass(q, kin, None, 0.6, np.zeros(B), np.array(lin))
    assert np.allclose(f1, 1.0, atol=1e-12) and np.allclose(o1, 1.0, atol=1e-12)
    fa, _ = orc.watched_mass(q, kin, kout, 0.6, np.zeros(B), np.array([20, 3, 8]))
    fb, _ = orc.watched_mass(q, kin, kout, 0.6, np.array([20, 3, 8]), np.array(lin))
    fall, _ = orc.watched_mass(q, kin, kout, 0.6, np.zeros(B), np.array(lin))
    assert np.allclose(fa + fb, fall, atol=1e-12)
    # uniform scores: the share is the fraction of tokens watched
    fu, ou = orc.watched_mass(np.zeros_like(q), kin, kout, 0.6, np.array([2, 2, 2]), np.array([12, 5, 10]))
    assert np.allclose(fu[:, 0], [10 / 49, 3 / 7, 8 / 19], atol=1e-12) and np.allclose(ou[:, 0], [10 / 40, 3 / 7, 8 / 16], atol=1e-12)


# ---------------------------------------------------------------- prefill: causal attention over the prompt
def test_prefill_is_causal_softmax_and_hands_over_to_decode():
    rng = np.random.default_rng(41)
    Hq, Hkv, D = 4, 2, 8
    lens = [37, 1, 20]
    ip = np.concatenate([[0], np.cumsum(lens)])
    T = int(ip[-1])
    q = rng.standard_normal((T, Hq, D)).astype(np.float32)
    k = rng.standard_normal((T, Hkv, D)).astype(np.float32)
    v = rng.standard_normal((T, Hkv, D)).astype(np.float32)
    y = orc.prefill(q, k, v, ip, 0.45)
    # textbook: per user, lower-triangular mask, softmax, times V (dense NumPy, float64)
    for u, L in enumerate(lens):
        a = int(ip[u])
        for h in range(Hq):
            S = 0.45 * q[a:a + L, h].astype(np.float64) @ k[a:a + L, h // 2].astype(np.float64).T
            S = np.where(np.tril(np.ones((L, L), bool)), S, -np.inf)
            Pm = np.exp(S - S.max(1, keepdims=True))
            Pm /= Pm.sum(1, keepdims=True)
            assert np.max(np.abs(y[a:a + L, h] - Pm @ v[a:a + L, h // 2].astype(np.float64))) < 1e-12
        assert np.array_equal(y[a, 0], v[a, 0].astype(np.float64))          # the first token sees only itself
    # the listed-rows form agrees with the full form
    rows = np.array([0, 5, 36, 37, 38, 57])
    assert np.array_equal(orc.prefill(q, k, v, ip, 0.45, rows), y[rows])
    # hand-over: store the prompt's K/V in a paged cache; a decode query equal to the last prompt token's q
    # must reproduce that token's prefill output (it attends to the same keys)
    ks = [np.zeros((Hkv, L, D), np.float32) for L in lens]
    kv = dense_to_paged(ks, ks, rng=rng)
    kv.seq_lens[:] = 0
    orc.write_prompt_kv(kv, k, v, ip)
    assert kv.seq_lens.tolist() == lens
    last = ip[1:] - 1
    yd = orc.full(q[last], kv, None, 0.45)
    assert np.max(np.abs(yd - y[last])) < 1e-12
