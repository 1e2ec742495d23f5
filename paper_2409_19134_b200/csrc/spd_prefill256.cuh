// Prefill for long prompts: the same causal attention as prefill_kernel, with 256 query rows per CTA.
//
// prefill_kernel is bound by shared-memory bandwidth: every 128 x 64 x 16 MMA streams 6 KB of operands
// for 32 cycles of math, and every K/V block is written to shared memory once per 128 query rows.
// Here one CTA owns the whole SM and two 128-row query tiles, and walks 128-key blocks:
//     S_t = Q_t K^T        128 x 128 x head_dim  (8 KB of operands per 64 cycles of math)
//     O_t += P_t V         128 x head_dim x 128, P_t read from tensor memory
// so each K/V block is loaded once for 256 query rows and a block's operand traffic drops by a third.
// Tensor memory: S_0, S_1 at columns [0, 128) and [128, 256); O_0, O_1 at [256, 384) and [384, 512);
// P_t (bf16 pairs, 64 columns) overwrites the upper half of S_t once the scores are in registers.
// Each tile has ONE S buffer, so within a tile the steps alternate (S, softmax, P V, next S); the two
// tiles run half a period apart: while the softmax warps of one tile work, the tensor core serves the other.
// Seventeen warps: sixteen do the softmax, two threads per query row (warp w and warp w ^ 8 share the
// rows of TMEM lane quarter w & 3 in tile (w >> 2) & 1; each takes 64 of a block's 128 keys and half of
// O's columns, and they exchange their row maxima through shared memory), so a tile's softmax takes about
// as long as the other tile's MMAs.  One thread of warp 16 issues every TMA load and every MMA.  Hand-over
// by mbarriers (and one named barrier per warp pair); every wait is bounded.
#pragma once

#include "spd_prefill.cuh"

namespace spd {

constexpr int kP2Rows = 256;                        // query rows per CTA (two tiles of 128)
constexpr int kP2Keys = 128;                        // keys per block
constexpr int kP2Box = 128 * 128;                   // one swizzled box: 128 rows x 128 bytes
constexpr int kP2Tile = 2 * kP2Box;                 // 128 rows x 128 channels
constexpr int kP2TmemCols = 512;
constexpr int kP2Threads = 544;

// Q x2, K x2, V x2, then eleven mbarriers and one word, then the row-maximum exchange [slot][tile][half][row].
constexpr size_t prefill256_smem_bytes() { return 6 * static_cast<size_t>(kP2Tile) + 128 + 2 * 2 * 2 * 128 * sizeof(float); }

__global__ void __launch_bounds__(kP2Threads, 1)
prefill256_kernel(const __grid_constant__ PrefillParams p, const __grid_constant__ CUtensorMap mq,
                  const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv) {
    extern __shared__ __align__(1024) uint8_t base[];
    const uint32_t Qs = smem_u32(base), Ks = Qs + 2 * kP2Tile, Vs = Ks + 2 * kP2Tile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + 6 * kP2Tile);
    uint64_t &bar_q = bars[0];
    uint64_t *bar_k = bars + 1, *bar_v = bars + 3;                         // K / V slot loaded
    uint64_t *bar_s = bars + 5, *bar_p = bars + 7, *bar_o = bars + 9;      // per tile: S ready, P written, O updated
    uint32_t &tmem_slot = *reinterpret_cast<uint32_t *>(bars + 11);
    float *xch = reinterpret_cast<float *>(base + 6 * kP2Tile + 128);
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / (p.Hq / p.Hkv);

    // which (user, 256-row query block) this CTA owns; heaviest blocks first.  Every warp finds it for itself.
    int qb = -1, first = 0, len = 0;
    {
        int blk = blockIdx.x;
        for (int u0 = 0; u0 < p.B; u0 += 32) {
            const int u = u0 + lane;
            int64_t a = 0, b = 0;
            if (u < p.B) { a = p.tok_indptr[u]; b = p.tok_indptr[u + 1]; }
            const bool bad = a < 0 || b < a || b > p.T;
            const int nb = bad ? 0 : static_cast<int>((b - a + kP2Rows - 1) / kP2Rows);
            int inc = nb;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += t;
            }
            const unsigned badmask = __ballot_sync(0xffffffffu, bad), hit = __ballot_sync(0xffffffffu, blk < inc);
            if (hit) {
                const int src = __ffs(hit) - 1;
                const int nb_s = __shfl_sync(0xffffffffu, nb, src), inc_s = __shfl_sync(0xffffffffu, inc, src);
                const int a_s = __shfl_sync(0xffffffffu, static_cast<int>(a), src), b_s = __shfl_sync(0xffffffffu, static_cast<int>(b), src);
                if (!(badmask & ((1u << src) - 1u))) { qb = nb_s - 1 - (blk - (inc_s - nb_s)); first = a_s; len = b_s - a_s; }
                break;
            }
            if (badmask) break;
            blk -= __shfl_sync(0xffffffffu, inc, 31);
        }
    }
    if (qb < 0) return;   // uniform over the CTA: no barrier, no TMEM touched yet
    // Tile t holds rows [256 qb + 128 t, + 128) and needs the 128-key blocks 0 .. 2 qb + t (the last one is
    // its diagonal).  The second tile may lie wholly past the prompt's end: then it is left out.
    const bool active1 = qb * kP2Rows + 128 < len;
    const int nkv0 = 2 * qb + 1, nkv1 = active1 ? 2 * qb + 2 : 0;
    const int NB = active1 ? nkv1 : nkv0;

    auto load_k = [&](int j) {
        const uint32_t bar = smem_u32(&bar_k[j & 1]);
        mbar_expect_tx(bar, kP2Tile);
        tma_load_3d(Ks + (j & 1) * kP2Tile, &mk, 0, kvh, first + j * kP2Keys, bar);
        tma_load_3d(Ks + (j & 1) * kP2Tile + kP2Box, &mk, 64, kvh, first + j * kP2Keys, bar);
    };
    auto load_v = [&](int j) {
        const uint32_t bar = smem_u32(&bar_v[j & 1]);
        mbar_expect_tx(bar, kP2Tile);
        tma_load_3d(Vs + (j & 1) * kP2Tile, &mv, 0, kvh, first + j * kP2Keys, bar);
        tma_load_3d(Vs + (j & 1) * kP2Tile + kP2Box, &mv, 64, kvh, first + j * kP2Keys, bar);
    };
    if (tid == 512) {     // the issuing thread sets the barriers up and starts the first loads before anything else happens
        for (int b = 0; b < 11; ++b) mbar_init(smem_u32(&bars[b]), (b == 7 || b == 8) ? 256 : 1);   // P written: a tile's softmax threads arrive
        fence_mbar_init();
        fence_proxy_async();
        const uint32_t bq = smem_u32(&bar_q);
        mbar_expect_tx(bq, active1 ? 2 * kP2Tile : kP2Tile);
        for (int t = 0; t < (active1 ? 2 : 1); ++t) {
            tma_load_3d(Qs + t * kP2Tile, &mq, 0, h, first + qb * kP2Rows + t * 128, bq);
            tma_load_3d(Qs + t * kP2Tile + kP2Box, &mq, 64, h, first + qb * kP2Rows + t * 128, bq);
        }
        load_k(0);
        load_v(0);
        if (NB > 1) { load_k(1); load_v(1); }
    }
    if (wid == 0) {       // one warp allocates all of tensor memory for the CTA (it has the SM to itself)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kP2TmemCols) : "memory");
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
    const int t = (wid >> 2) & 1;            // tile of a softmax warp
    const int half = (wid >> 3) & 1;         // which 64 keys of a block, and which 64 columns of O, this thread takes
    const int row = (wid & 3) * 32 + lane;   // query row of a softmax thread within its tile
    const int pair_bar = 1 + t * 4 + (wid & 3);   // named barrier of this warp and its partner (64 threads)
    const uint32_t t_lane = tmem + (static_cast<uint32_t>((wid & 3) * 32) << 16);   // this warp's 32 lanes
    const int nkv = t == 0 ? nkv0 : nkv1;

    if (wid == 16) {
        // ---------------- the issuing thread: TMA loads and MMAs ----------------------------------------
        if (tid == 512) {
            auto mma_s = [&](int tt, int j) {        // S_tt(j) = Q_tt K(j)^T, 16 channels per MMA
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t a = umma_desc(Qs + tt * kP2Tile + (kk >> 2) * kP2Box + (kk & 3) * 32, 16, 1024);
                    const uint64_t b = umma_desc(Ks + (j & 1) * kP2Tile + (kk >> 2) * kP2Box + (kk & 3) * 32, 16, 1024);
                    umma_bf16(tmem + tt * 128, a, b, umma_idesc(false, 128), kk > 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_s[tt]));
            };
            ok = mbar_wait(smem_u32(&bar_q), 0) && mbar_wait(smem_u32(&bar_k[0]), 0);
            mma_s(0, 0);
            if (active1) mma_s(1, 0);
            for (int j = 0; j < NB; ++j) {
                // V slot (j+1) & 1 held V(j-1): free once both tiles' O have taken block j-1 in (issued a round ago)
                if (j >= 1 && j + 1 < NB) {
                    if (j - 1 < nkv0) ok = mbar_wait(smem_u32(&bar_o[0]), (j - 1) & 1) && ok;
                    if (j - 1 < nkv1) ok = mbar_wait(smem_u32(&bar_o[1]), (j - 1) & 1) && ok;
                    load_v(j + 1);
                }
                for (int tt = 0; tt < 2; ++tt) {
                    if (j >= (tt == 0 ? nkv0 : nkv1)) continue;
                    ok = mbar_wait(smem_u32(&bar_p[tt]), j & 1) && ok;          // P_tt(j) written, O_tt rescaled
                    ok = mbar_wait(smem_u32(&bar_v[j & 1]), (j >> 1) & 1) && ok;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {   // O_tt += P_tt V(j), 16 keys per MMA; P from TMEM (8 columns per 16 keys; keys 0-63 at column 0, 64-127 at column 64)
                        // V is [key][channel]: MN-major for the B operand; 8-key groups 1024 bytes apart, 64-channel boxes one box apart
                        const uint64_t b = umma_desc(Vs + (j & 1) * kP2Tile + kk * 2048, kP2Box, 1024);
                        umma_bf16_ta(tmem + 256 + tt * 128, tmem + tt * 128 + (kk >> 2) * 64 + (kk & 3) * 8, b, umma_idesc(true, 128), (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bar_o[tt]));
                    // S_tt(j+1) overwrites S_tt(j) / P_tt(j): the MMAs above were issued first, so they run first
                    if (j + 1 < (tt == 0 ? nkv0 : nkv1)) {
                        ok = mbar_wait(smem_u32(&bar_k[(j + 1) & 1]), ((j + 1) >> 1) & 1) && ok;
                        mma_s(tt, j + 1);
                    }
                }
                // K slot j & 1: both tiles' S(j) exist (their P(j) was seen) and S(j+1) reads the other slot
                if (j + 2 < NB) load_k(j + 2);
            }
            ok = mbar_wait(smem_u32(&bar_o[0]), (nkv0 - 1) & 1) && ok;
            if (active1) ok = mbar_wait(smem_u32(&bar_o[1]), (nkv1 - 1) & 1) && ok;
        }
    } else if (nkv > 0) {
        // ---------------- softmax warps: one query row per thread -------------------------------------------
        const float c2 = p.sm_scale * kLog2e;    // scores in log2 units
        const uint32_t tS = t_lane + t * 128 + half * 64, tOt = t_lane + 256 + t * 128 + half * 64;
        float m = -INFINITY;
        for (int j = 0; j < nkv; ++j) {
            ok = mbar_wait(smem_u32(&bar_s[t]), j & 1) && ok;                      // S_t(j) is there
            tc_fence_after();
            float sv[64];
            tmem_ld64(tS, sv);
            // only the last block (the tile's diagonal) hides anything: key column i is visible iff i <= row
            if (j == nkv - 1) {
                const int ahead = row + 1 - half * 64;
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
            // the row's maximum over all 128 keys: swap halves with the partner thread (two slots, so that a
            // fast thread's next block cannot overwrite what its partner has yet to read)
            float rmax = fmaxf(fmax3(r4[0], r4[1], r4[2]), r4[3]);
            float *slot = xch + (j & 1) * 512 + t * 256;
            slot[half * 128 + row] = rmax;
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            rmax = fmaxf(rmax, slot[(half ^ 1) * 128 + row]) * c2;   // finite from the first block on: key 0 is visible to every row
            // m is a reference point in log2 units of the scaled score that moves only when the block's
            // maximum lies more than kPfSlack above it (see prefill_kernel); both partners decide alike
            const float m_new = (rmax > m + kPfSlack) ? rmax : m;
            const float alpha = ex2_approx(m - m_new);
            const uint64_t c2x2 = pack_f32x2(c2, c2), mx2 = pack_f32x2(-m_new, -m_new);
            uint64_t lsum2 = 0;                           // two partial row sums, (+0, +0)
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 64; i += 2) {
                float a0, a1;
                unpack_f32x2(fma_f32x2(pack_f32x2(sv[i], sv[i + 1]), c2x2, mx2), a0, a1);
                const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                lsum2 = add_f32x2(lsum2, pack_f32x2(p0, p1));
                pk[i >> 1] = pack_bf16(p0, p1);
            }
            // this half of P_t(j) as bf16 pairs over the first 32 of the columns this thread read: the A operand
            // of O += P V (row = lane, two keys per column)
            tmem_st32u(tS, pk);
            {
                float s0, s1;
                unpack_f32x2(lsum2, s0, s1);
                l = l * alpha + (s0 + s1);                // this thread's half of the row sum
            }
            m = m_new;
            // rescale this thread's half of O where the reference moved (rare): only then must
            // O += P(j-1) V(j-1) have finished
            if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
                ok = mbar_wait(smem_u32(&bar_o[t]), (j - 1) & 1) && ok;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    float ov[32];
                    tmem_ld32(tOt + c * 32, ov);
#pragma unroll
                    for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                    tmem_st32(tOt + c * 32, ov);
                }
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bar_p[t]));
        }
        ok = mbar_wait(smem_u32(&bar_o[t]), (nkv - 1) & 1) && ok;
    }
    tc_fence_after();
    const bool gave_up = !__syncthreads_and(ok);
    if (gave_up) {
        if (tid == 0) flag_error(p.hdr, 6 /* SPD_ERR_TIMEOUT */, -1);
    } else if (wid < 16 && nkv > 0) {
        // ---- the row sum is the two partners' halves together; then each thread normalises its 64 channels
        //      into shared memory (the tile's own Q is free: all its MMAs are done), and the warps store whole
        //      rows (16-byte chunks XOR-swizzled by the row against bank conflicts); rows past the prompt's end
        //      are not stored
        float *slot = xch + t * 256;
        slot[half * 128 + row] = l;
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        const float inv = 1.f / (l + slot[(half ^ 1) * 128 + row]);
        uint8_t *stage = base + t * kP2Tile;                    // 128 rows x 256 bytes
        const uint32_t tOt = t_lane + 256 + t * 128 + half * 64;
        const int rows_live = len - (qb * kP2Rows + t * 128 + (wid & 3) * 32);   // rows of this warp that belong to the prompt
        const int64_t tok0 = static_cast<int64_t>(first) + qb * kP2Rows + t * 128 + (wid & 3) * 32;
        uint8_t *dst = reinterpret_cast<uint8_t *>(p.out);
        if (p.out_bf16) {
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                float ov[32];
                tmem_ld32(tOt + c * 32, ov);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<uint4 *>(stage + row * 256 + (((half * 8 + c * 4 + q4) ^ (row & 7)) << 4)) =
                        make_uint4(pack_bf16(ov[8 * q4] * inv, ov[8 * q4 + 1] * inv), pack_bf16(ov[8 * q4 + 2] * inv, ov[8 * q4 + 3] * inv),
                                   pack_bf16(ov[8 * q4 + 4] * inv, ov[8 * q4 + 5] * inv), pack_bf16(ov[8 * q4 + 6] * inv, ov[8 * q4 + 7] * inv));
            }
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            // each partner stores 16 of the pair's 32 rows, two rows per instruction
#pragma unroll 4
            for (int it = 0; it < 8; ++it) {
                const int r = half * 16 + 2 * it + (lane >> 4), ch = lane & 15, rr = (wid & 3) * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 256 + ch * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 7)) << 4));
            }
        } else {
            // fp32 rows are 512 bytes: the partner with channels 0-63 goes first, then the other, through the same 256-byte lines
            if (half == 1) asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                float ov[32];
                tmem_ld32(tOt + c * 32, ov);
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4)
                    *reinterpret_cast<float4 *>(stage + row * 256 + (((c * 8 + q4) ^ (row & 7)) << 4)) =
                        make_float4(ov[4 * q4] * inv, ov[4 * q4 + 1] * inv, ov[4 * q4 + 2] * inv, ov[4 * q4 + 3] * inv);
            }
            __syncwarp();
#pragma unroll 4
            for (int it = 0; it < 16; ++it) {
                const int r = 2 * it + (lane >> 4), ch = lane & 15, rr = (wid & 3) * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 512 + half * 256 + ch * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 7)) << 4));
            }
            if (half == 0) asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kP2TmemCols) : "memory");
}

}  // namespace spd
