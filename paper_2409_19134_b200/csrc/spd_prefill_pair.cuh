// Prefill for long prompts: prefill_kernel's pipeline twice in one CTA, over shared K/V blocks.
//
// With every SM running two independent prefill_kernel CTAs, each K/V block crosses from L2 to shared
// memory once per 128 query rows, and that traffic (about 7 TB/s at 950 TFLOP/s) together with its
// latency is what holds the kernel back: taking the K/V loads out (scratch copy) made it 28 % faster.
// Here one CTA has the SM to itself and owns TWO 128-row query tiles of the same (user, head); the 64-key
// K/V blocks are loaded once for both, into four-slot rings (as much shared memory as before, twice the
// look-ahead).  Per tile everything is as in prefill_kernel: S = Q_t K^T into two TMEM buffers, softmax with
// one row per thread, P back into S's columns, O_t += P V from TMEM, one thread issuing the S products and one
// the P V products.  Tile t uses TMEM columns [256 t, 256 t + 256): S buffers at +0 and +64, O at +128.
// Thirteen warps: 0-3 and 4-7 softmax of tile 0 and 1; 8 / 9 the issuing threads of tile 0 (S / P V);
// 10 / 11 those of tile 1; 12 the thread that loads, refilling a ring slot when the tensor core has
// released it for both tiles (tcgen05.commit on a "slot free" barrier that counts the tiles).
// Hand-over by mbarriers only; every wait is bounded.
#pragma once

#include "spd_prefill.cuh"

namespace spd {

constexpr int kPpRows = 256;                        // query rows per CTA (two tiles of 128)
constexpr int kPpSlots = 4;                         // K and V ring depth
constexpr int kPpTmemCols = 512;
constexpr int kPpThreads = 416;
constexpr int kPpBars = 1 + 12 + 4 * kPpSlots;      // Q; per tile S, P, O twice; per slot K, V loaded and K, V free

// Q x2, K x4, V x4, then the mbarriers and one word.
constexpr size_t prefill_pair_smem_bytes() { return 2 * kPfQTile + 2 * kPpSlots * static_cast<size_t>(kPfKvTile) + 256; }
static_assert(kPpBars * 8 + 4 <= 256, "barrier block");

__global__ void __launch_bounds__(kPpThreads, 1)
prefill_pair_kernel(const __grid_constant__ PrefillParams p, const __grid_constant__ CUtensorMap mq,
                    const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv) {
    extern __shared__ __align__(1024) uint8_t base[];
    const uint32_t Qs = smem_u32(base), Ks = Qs + 2 * kPfQTile, Vs = Ks + kPpSlots * kPfKvTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + 2 * kPfQTile + 2 * kPpSlots * kPfKvTile);
    uint64_t &bar_q = bars[0];
    uint64_t *bar_s = bars + 1, *bar_p = bars + 5, *bar_o = bars + 9;      // [tile][S buffer]: S ready, P written, O updated
    uint64_t *bar_k = bars + 13, *bar_v = bar_k + kPpSlots;                // ring slot loaded
    uint64_t *bar_kfree = bar_v + kPpSlots, *bar_vfree = bar_kfree + kPpSlots;   // ring slot read by every tile that needs it
    uint32_t &tmem_slot = *reinterpret_cast<uint32_t *>(bars + kPpBars);
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / (p.Hq / p.Hkv);

    if (tid == 384) { prefetch_tensormap(&mq); prefetch_tensormap(&mk); prefetch_tensormap(&mv); }   // needed right after the search below
    int qb, first, len;
    prefill_find_block(p, kPpRows, blockIdx.x, lane, qb, first, len);
    if (qb < 0) return;   // uniform over the CTA: no barrier, no TMEM touched yet
    // Tile t holds rows [256 qb + 128 t, + 128) and needs the 64-key blocks 0 .. 4 qb + 2 t + 1 (the last two
    // straddle its diagonal).  The second tile may lie wholly past the prompt's end: then it is left out.
    const bool active1 = qb * kPpRows + 128 < len;
    const int nkv0 = 4 * qb + 2, nkv1 = active1 ? 4 * qb + 4 : 0;
    const int NB = active1 ? nkv1 : nkv0;

    auto load_k = [&](int j) {
        const uint32_t bar = smem_u32(&bar_k[j % kPpSlots]);
        mbar_expect_tx(bar, kPfKvTile);
        tma_load_3d(Ks + (j % kPpSlots) * kPfKvTile, &mk, 0, kvh, first + j * kPfKeys, bar);
        tma_load_3d(Ks + (j % kPpSlots) * kPfKvTile + kPfKvBox, &mk, 64, kvh, first + j * kPfKeys, bar);
    };
    auto load_v = [&](int j) {
        const uint32_t bar = smem_u32(&bar_v[j % kPpSlots]);
        mbar_expect_tx(bar, kPfKvTile);
        tma_load_3d(Vs + (j % kPpSlots) * kPfKvTile, &mv, 0, kvh, first + j * kPfKeys, bar);
        tma_load_3d(Vs + (j % kPpSlots) * kPfKvTile + kPfKvBox, &mv, 64, kvh, first + j * kPfKeys, bar);
    };
    if (tid == 384) {     // the loading thread sets the barriers up and starts the first loads before anything else happens
        for (int b = 0; b < kPpBars; ++b)     // P written: one arrival per softmax warp of the tile; slot free: one commit per tile
            mbar_init(smem_u32(&bars[b]), (b >= 5 && b < 9) ? 4 : (b >= 13 + 2 * kPpSlots ? (active1 ? 2 : 1) : 1));
        fence_mbar_init();
        fence_proxy_async();
        const uint32_t bq = smem_u32(&bar_q);
        mbar_expect_tx(bq, active1 ? 2 * kPfQTile : kPfQTile);
        for (int t = 0; t < (active1 ? 2 : 1); ++t) {
            tma_load_3d(Qs + t * kPfQTile, &mq, 0, h, first + qb * kPpRows + t * 128, bq);
            tma_load_3d(Qs + t * kPfQTile + kPfQBox, &mq, 64, h, first + qb * kPpRows + t * 128, bq);
        }
        for (int j = 0; j < kPpSlots && j < NB; ++j) { load_k(j); load_v(j); }
    }
    if (wid == 0) {       // one warp allocates all of tensor memory for the CTA (it has the SM to itself)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kPpTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    // Every wait is bounded.  A wait that runs out clears `ok` and the thread carries on (with garbage, but
    // towards the same end): nothing in the loop waits for all threads, so nobody can be left behind.
    bool ok = true;
    float l = 0.f;
    const int t = wid < 8 ? (wid >> 2) : ((wid - 8) >> 1) & 1;   // tile of a softmax warp (0-7) or of an issuing warp (8-11)
    const int nkv = t == 0 ? nkv0 : nkv1;
    const int row = tid & 127;                                     // query row of a softmax thread within its tile
    const uint32_t tT = tmem + t * 256;                            // this tile's columns: S buffers at +0 and +64, O at +128
    const uint32_t t_lane = tT + (static_cast<uint32_t>((wid & 3) * 32) << 16);   // a softmax warp's 32 lanes
    uint64_t *bs = bar_s + 2 * t, *bp = bar_p + 2 * t, *bo = bar_o + 2 * t;

    if (wid == 12) {
        // ---------------- the loading thread: block j + 4 goes where block j was, once every tile is done with it
        if (tid == 384) {
            for (int j = 0; j + kPpSlots < NB; ++j) {
                ok = mbar_wait(smem_u32(&bar_kfree[j % kPpSlots]), (j / kPpSlots) & 1) && ok;
                load_k(j + kPpSlots);
                ok = mbar_wait(smem_u32(&bar_vfree[j % kPpSlots]), (j / kPpSlots) & 1) && ok;
                load_v(j + kPpSlots);
            }
        }
    } else if (wid >= 8) {
        if (lane == 0 && nkv > 0) {
            if (((wid - 8) & 1) == 0) {
                // ---------------- a tile's first issuing thread: S = Q_t K^T ------------------------------------
                auto mma_s = [&](int j) {            // S(j) into S buffer j & 1; 16 channels per MMA
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint64_t a = umma_desc(Qs + t * kPfQTile + (kk >> 2) * kPfQBox + (kk & 3) * 32, 16, 1024);
                        const uint64_t b = umma_desc(Ks + (j % kPpSlots) * kPfKvTile + (kk >> 2) * kPfKvBox + (kk & 3) * 32, 16, 1024);
                        umma_bf16(tT + (j & 1) * kPfKeys, a, b, umma_idesc(false, kPfKeys), kk > 0 ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bs[j & 1]));
                    umma_commit(smem_u32(&bar_kfree[j % kPpSlots]));
                };
                ok = mbar_wait(smem_u32(&bar_q), 0) && mbar_wait(smem_u32(&bar_k[0]), 0);
                mma_s(0);
                for (int j = 0; j + 1 < nkv; ++j) {
                    ok = mbar_wait(smem_u32(&bar_k[(j + 1) % kPpSlots]), ((j + 1) / kPpSlots) & 1) && ok;
                    // S(j+1) goes where S(j-1) and then P(j-1) were: free once O has taken block j-1 in (the other
                    // thread's MMAs: wait for their commit)
                    if (j > 0) ok = mbar_wait(smem_u32(&bo[(j - 1) & 1]), ((j - 1) >> 1) & 1) && ok;
                    mma_s(j + 1);
                }
            } else {
                // ---------------- a tile's second issuing thread: O_t += P V --------------------------------------
                for (int j = 0; j < nkv; ++j) {
                    ok = mbar_wait(smem_u32(&bp[j & 1]), (j >> 1) & 1) && ok;          // P(j) is written and O rescaled
                    ok = mbar_wait(smem_u32(&bar_v[j % kPpSlots]), (j / kPpSlots) & 1) && ok;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {   // 16 keys per MMA; P comes from TMEM (8 columns per 16 keys)
                        // V is [key][channel]: MN-major for the B operand; 8-key groups 1024 bytes apart, 64-channel boxes one box apart
                        const uint64_t b = umma_desc(Vs + (j % kPpSlots) * kPfKvTile + kk * 2048, kPfKvBox, 1024);
                        umma_bf16_ta(tT + 128, tT + (j & 1) * kPfKeys + kk * 8, b, umma_idesc(true, 128), (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bo[j & 1]));
                    umma_commit(smem_u32(&bar_vfree[j % kPpSlots]));
                }
                ok = mbar_wait(smem_u32(&bo[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
            }
        }
    } else if (nkv > 0) {
        // ---------------- softmax warps: one query row per thread -------------------------------------------
        const float c2 = p.sm_scale * kLog2e;    // scores in log2 units
        float m = -INFINITY;
        for (int j = 0; j < nkv; ++j) {
            ok = mbar_wait(smem_u32(&bs[j & 1]), (j >> 1) & 1) && ok;              // S(j) is there
            tc_fence_after();
            float sv[64];
            tmem_ld64(t_lane + (j & 1) * kPfKeys, sv);
            // only the tile's last two blocks (on its diagonal) hide anything; `ahead` = first column of this
            // block that lies ahead of this row
            if (j >= nkv - 2) {
                const int ahead = (128 * (2 * qb + t) + row) - kPfKeys * j + 1;
#pragma unroll
                for (int i = 0; i < 64; ++i) sv[i] = (i >= ahead) ? -INFINITY : sv[i];
            }
            float r4[4];                                 // four chains of three-input maxima
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                r4[c] = fmax3(sv[16 * c], sv[16 * c + 1], sv[16 * c + 2]);
#pragma unroll
                for (int i = 3; i < 15; i += 2) r4[c] = fmax3(r4[c], sv[16 * c + i], sv[16 * c + i + 1]);
                r4[c] = fmaxf(r4[c], sv[16 * c + 15]);
            }
            // m is a reference point in log2 units of the scaled score that moves only when the block's
            // maximum lies more than kPfSlack above it (see prefill_kernel)
            const float rmax = fmaxf(fmax3(r4[0], r4[1], r4[2]), r4[3]) * c2;   // finite from the first block on: key 0 is visible to every row
            const float m_new = (rmax > m + kPfSlack) ? rmax : m;
            const float alpha = ex2_approx(m - m_new);
            uint32_t pk[32];
            const uint64_t c2x2 = pack_f32x2(c2, c2), mx2 = pack_f32x2(-m_new, -m_new);
            uint64_t lsum2 = 0;                           // two partial row sums, (+0, +0)
#pragma unroll
            for (int i = 0; i < 64; i += 2) {
                float a0, a1;
                unpack_f32x2(fma_f32x2(pack_f32x2(sv[i], sv[i + 1]), c2x2, mx2), a0, a1);
                const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                lsum2 = add_f32x2(lsum2, pack_f32x2(p0, p1));
                pk[i >> 1] = pack_bf16(p0, p1);
            }
            {
                float s0, s1;
                unpack_f32x2(lsum2, s0, s1);
                l = l * alpha + (s0 + s1);
            }
            m = m_new;
            // rescale O where the reference moved (rare): only then must O += P(j-1) V(j-1) have finished
            if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
                ok = mbar_wait(smem_u32(&bo[(j - 1) & 1]), ((j - 1) >> 1) & 1) && ok;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float ov[32];
                    tmem_ld32(t_lane + 128 + c * 32, ov);
#pragma unroll
                    for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                    tmem_st32(t_lane + 128 + c * 32, ov);
                }
            }
            // P(j) as bf16 pairs over the first 32 columns of S(j)'s buffer: the A operand of O += P V
            tmem_st32u(t_lane + (j & 1) * kPfKeys, pk);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();                                 // one arrival per warp
            if (lane == 0) mbar_arrive(smem_u32(&bp[j & 1]));
        }
        ok = mbar_wait(smem_u32(&bo[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
    }
    tc_fence_after();
    const bool gave_up = !__syncthreads_and(ok);
    if (gave_up) {
        if (tid == 0) flag_error(p.hdr, 6 /* SPD_ERR_TIMEOUT */, -1);
    } else if (wid < 8 && nkv > 0) {
        // ---- normalise this thread's row into shared memory (the tile's own Q is free: all its MMAs are
        //      done), 256 bytes of a row at a time, then each warp stores its own 32 rows, two rows per
        //      instruction; 16-byte chunks are XOR-swizzled by the row against bank conflicts; rows past the
        //      prompt's end are not stored
        const float inv = 1.f / l;
        uint8_t *stage = base + t * kPfQTile;                   // 128 rows x 256 bytes
        const int rows_live = len - (qb * kPpRows + t * 128 + (wid & 3) * 32);   // rows of this warp that belong to the prompt
        const int64_t tok0 = static_cast<int64_t>(first) + qb * kPpRows + t * 128 + (wid & 3) * 32;
        uint8_t *dst = reinterpret_cast<uint8_t *>(p.out);
        const int passes = p.out_bf16 ? 1 : 2, row_bytes = p.out_bf16 ? 256 : 512;
#pragma unroll 1
        for (int pass = 0; pass < passes; ++pass) {             // fp32: channels [64 pass, 64 pass + 64)
            if (p.out_bf16) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float ov[32];
                    tmem_ld32(t_lane + 128 + c * 32, ov);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        *reinterpret_cast<uint4 *>(stage + row * 256 + (((c * 4 + q4) ^ (row & 7)) << 4)) =
                            make_uint4(pack_bf16(ov[8 * q4] * inv, ov[8 * q4 + 1] * inv), pack_bf16(ov[8 * q4 + 2] * inv, ov[8 * q4 + 3] * inv),
                                       pack_bf16(ov[8 * q4 + 4] * inv, ov[8 * q4 + 5] * inv), pack_bf16(ov[8 * q4 + 6] * inv, ov[8 * q4 + 7] * inv));
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    float ov[32];
                    tmem_ld32(t_lane + 128 + pass * 64 + c * 32, ov);
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        *reinterpret_cast<float4 *>(stage + row * 256 + (((c * 8 + q4) ^ (row & 7)) << 4)) =
                            make_float4(ov[4 * q4] * inv, ov[4 * q4 + 1] * inv, ov[4 * q4 + 2] * inv, ov[4 * q4 + 3] * inv);
                }
            }
            __syncwarp();
#pragma unroll 4
            for (int it = 0; it < 16; ++it) {
                const int r = 2 * it + (lane >> 4), ch = lane & 15, rr = (wid & 3) * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * row_bytes + pass * 256 + ch * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 7)) << 4));
            }
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPpTmemCols) : "memory");
}

}  // namespace spd
