// Prefill for long prompts: the same causal attention as prefill_kernel, walking 128-key blocks.
//
// What bounds prefill_kernel is the tensor core's instruction rate: a 128 x 64 x 16 MMA occupies it for
// about twice as long as its 32 cycles of math, a 128 x 128 x 16 MMA for little more than its 64.  So here
// both products use N = 128:
//     S = Q K^T            128 x 128 x head_dim   -> TMEM, two buffers: columns [0, 128) and [128, 256)
//     O += P V             128 x head_dim x 128   -> TMEM columns [256, 384); P read from TMEM
// That takes 384 TMEM columns and 160 KB of shared memory (Q, two K and two V blocks of 128 keys), so one
// CTA has the SM to itself, and the softmax, which two co-resident CTAs used to hide behind each other, has
// to keep up by itself: sixteen softmax warps, FOUR threads per query row.  Warp w works on the rows of TMEM
// lane quarter w & 3 and, of every block, on keys [32 (w >> 2), + 32) and on the same columns of O; the four
// threads of a row exchange their maxima through shared memory (one named barrier per lane quarter).  P goes
// back as bf16 pairs over the first 16 of the 32 columns each thread read.
// Two more warps hold one issuing thread each: S products and TMA loads / P V products (one thread cannot
// issue MMAs fast enough, see prefill_kernel).  Hand-over by mbarriers; every wait is bounded.
#pragma once

#include "spd_prefill.cuh"

namespace spd {

constexpr int kPwKeys = 128;                        // keys per block
constexpr int kPwBox = 128 * 128;                   // one swizzled box: 128 rows x 128 bytes
constexpr int kPwTile = 2 * kPwBox;                 // 128 rows x 128 channels
constexpr int kPwTmemCols = 512;                    // 384 used; the allocator hands out powers of two
constexpr int kPwThreads = 576;                     // 16 softmax warps + 2 warps with one issuing thread each

// Q, K x2, V x2, then eleven mbarriers and one word, then the exchange of row maxima [slot][part][row].
constexpr size_t prefill_wide_smem_bytes() { return 5 * static_cast<size_t>(kPwTile) + 128 + 2 * 4 * 128 * sizeof(float); }

__device__ __forceinline__ void tmem_st16u(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr),
          "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}

__global__ void __launch_bounds__(kPwThreads, 1)
prefill_wide_kernel(const __grid_constant__ PrefillParams p, const __grid_constant__ CUtensorMap mq,
                    const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv) {
    extern __shared__ __align__(1024) uint8_t base[];
    const uint32_t Qs = smem_u32(base), Ks = Qs + kPwTile, Vs = Ks + 2 * kPwTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + 5 * kPwTile);
    uint64_t &bar_q = bars[0];                                             // Q loaded
    uint64_t *bar_o = bars + 1;                                            // O has taken in the block whose P was in S buffer 0 / 1
    uint64_t *bar_p = bars + 3;                                            // P written into S buffer 0 / 1
    uint64_t *bar_k = bars + 5, *bar_v = bars + 7, *bar_s = bars + 9;     // K / V slot loaded; S buffer ready
    uint32_t &tmem_slot = *reinterpret_cast<uint32_t *>(bars + 11);
    float *xch = reinterpret_cast<float *>(base + 5 * kPwTile + 128);
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / (p.Hq / p.Hkv);

    // which (user, query block) this CTA owns; the heaviest blocks (closest to the prompt's end) come first.
    // Every warp works it out for itself, 32 users at a time.
    int qb = -1, first = 0, len = 0;
    {
        int blk = blockIdx.x;
        for (int u0 = 0; u0 < p.B; u0 += 32) {
            const int u = u0 + lane;
            int64_t a = 0, b = 0;
            if (u < p.B) { a = p.tok_indptr[u]; b = p.tok_indptr[u + 1]; }
            const bool bad = a < 0 || b < a || b > p.T;                   // inconsistent offsets: nothing from here on
            const int nb = bad ? 0 : static_cast<int>((b - a + kPfBlock - 1) / kPfBlock);
            int inc = nb;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += up;
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
    const int nkv = qb + 1;   // 128-key blocks up to and including the diagonal one

    auto load_k = [&](int j) {
        const uint32_t bar = smem_u32(&bar_k[j & 1]);
        mbar_expect_tx(bar, kPwTile);
        tma_load_3d(Ks + (j & 1) * kPwTile, &mk, 0, kvh, first + j * kPwKeys, bar);
        tma_load_3d(Ks + (j & 1) * kPwTile + kPwBox, &mk, 64, kvh, first + j * kPwKeys, bar);
    };
    auto load_v = [&](int j) {
        const uint32_t bar = smem_u32(&bar_v[j & 1]);
        mbar_expect_tx(bar, kPwTile);
        tma_load_3d(Vs + (j & 1) * kPwTile, &mv, 0, kvh, first + j * kPwKeys, bar);
        tma_load_3d(Vs + (j & 1) * kPwTile + kPwBox, &mv, 64, kvh, first + j * kPwKeys, bar);
    };
    if (tid == 512) {     // the first issuing thread sets the barriers up and starts the first loads before anything else happens
        for (int b = 0; b < 11; ++b) mbar_init(smem_u32(&bars[b]), (b == 3 || b == 4) ? 16 : 1);   // P written: one arrival per softmax warp
        fence_mbar_init();
        fence_proxy_async();
        const uint32_t bq = smem_u32(&bar_q);
        mbar_expect_tx(bq, kPwTile);
        tma_load_3d(Qs, &mq, 0, h, first + qb * kPfBlock, bq);
        tma_load_3d(Qs + kPwBox, &mq, 64, h, first + qb * kPfBlock, bq);
        load_k(0);
        load_v(0);
        if (nkv > 1) { load_k(1); load_v(1); }
    }
    if (wid == 0) {       // one warp allocates the accumulator columns for the CTA (it has the SM to itself)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kPwTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tO = tmem + 256;

    // Every mbarrier wait is bounded.  A wait that runs out clears `ok` and the thread carries on (with garbage,
    // but towards the same end); the named barriers are between warps that run the same number of rounds.
    bool ok = true;
    float l = 0.f;
    const int quarter = wid & 3;             // TMEM lane quarter of a softmax warp
    const int part = (wid >> 2) & 3;         // which 32 keys of a block, and which 32 columns of O, this thread takes
    const int row = quarter * 32 + lane;     // query row of a softmax thread within the block
    const int quad_bar = 1 + quarter;        // named barrier of the four warps that share these rows (128 threads)
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);   // this warp's 32 lanes

    if (wid == 16) {
        // ---------------- first issuing thread: TMA loads and S = Q K^T -------------------------------------
        if (tid == 512) {
            auto mma_s = [&](int j) {                // S(j) = Q K(j)^T into S buffer j & 1; 16 channels per MMA
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t a = umma_desc(Qs + (kk >> 2) * kPwBox + (kk & 3) * 32, 16, 1024);
                    const uint64_t b = umma_desc(Ks + (j & 1) * kPwTile + (kk >> 2) * kPwBox + (kk & 3) * 32, 16, 1024);
                    umma_bf16(tmem + (j & 1) * 128, a, b, umma_idesc(false, 128), kk > 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_s[j & 1]));
            };
            ok = mbar_wait(smem_u32(&bar_q), 0) && mbar_wait(smem_u32(&bar_k[0]), 0);
            mma_s(0);
            for (int j = 0; j < nkv; ++j) {
                if (j + 1 < nkv) {
                    ok = mbar_wait(smem_u32(&bar_k[(j + 1) & 1]), ((j + 1) >> 1) & 1) && ok;
                    // S(j+1) goes where S(j-1) and then P(j-1) were, and V(j+1) where V(j-1) was: both are free
                    // once O has taken block j-1 in (the other thread's MMAs: wait for their commit)
                    if (j > 0) ok = mbar_wait(smem_u32(&bar_o[(j - 1) & 1]), ((j - 1) >> 1) & 1) && ok;
                    mma_s(j + 1);
                    if (j > 0) load_v(j + 1);
                }
                if (j + 2 < nkv) {                     // K slot j & 1 is free once S(j) exists (issued a round ago)
                    ok = mbar_wait(smem_u32(&bar_s[j & 1]), (j >> 1) & 1) && ok;
                    load_k(j + 2);
                }
            }
        }
    } else if (wid == 17) {
        // ---------------- second issuing thread: O += P V -----------------------------------------------------
        if (tid == 544) {
            for (int j = 0; j < nkv; ++j) {
                ok = mbar_wait(smem_u32(&bar_p[j & 1]), (j >> 1) & 1) && ok;       // P(j) is written and O rescaled
                ok = mbar_wait(smem_u32(&bar_v[j & 1]), (j >> 1) & 1) && ok;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {       // 16 keys per MMA; P from TMEM: 8 columns per 16 keys, 32 keys per 32-column part
                    // V is [key][channel]: MN-major for the B operand; 8-key groups 1024 bytes apart, 64-channel boxes one box apart
                    const uint64_t b = umma_desc(Vs + (j & 1) * kPwTile + kk * 2048, kPwBox, 1024);
                    umma_bf16_ta(tO, tmem + (j & 1) * 128 + (kk >> 1) * 32 + (kk & 1) * 8, b, umma_idesc(true, 128), (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_o[j & 1]));
            }
            ok = mbar_wait(smem_u32(&bar_o[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
        }
    } else {
        // ---------------- softmax warps: four threads per query row -----------------------------------------
        const float c2 = p.sm_scale * kLog2e;    // scores in log2 units
        float m = -INFINITY;
        for (int j = 0; j < nkv; ++j) {
            const uint32_t tS = t_lane + (j & 1) * 128 + part * 32;
            ok = mbar_wait(smem_u32(&bar_s[j & 1]), (j >> 1) & 1) && ok;           // S(j) is there
            tc_fence_after();
            float sv[32];
            tmem_ld32(tS, sv);
            // only the last block (the diagonal) hides anything: key column i of the block is visible iff i <= row
            if (j == nkv - 1) {
                const int ahead = row + 1 - part * 32;
#pragma unroll
                for (int i = 0; i < 32; ++i) sv[i] = (i >= ahead) ? -INFINITY : sv[i];
            }
            float r2[2];                                 // two chains of three-input maxima
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                r2[c] = fmax3(sv[16 * c], sv[16 * c + 1], sv[16 * c + 2]);
#pragma unroll
                for (int i = 3; i < 15; i += 2) r2[c] = fmax3(r2[c], sv[16 * c + i], sv[16 * c + i + 1]);
                r2[c] = fmaxf(r2[c], sv[16 * c + 15]);
            }
            // the row's maximum over all 128 keys: through shared memory with the three other threads of the row
            // (two slots, so that a fast thread's next block cannot overwrite what another has yet to read)
            float rmax = fmaxf(r2[0], r2[1]);
            float *slot = xch + (j & 1) * 512;
            slot[part * 128 + row] = rmax;
            asm volatile("bar.sync %0, 128;" ::"r"(quad_bar) : "memory");
            rmax = fmaxf(fmaxf(slot[row], slot[128 + row]), fmaxf(slot[256 + row], slot[384 + row])) * c2;   // finite from the first block on: key 0 is visible to every row
            // m is a reference point in log2 units of the scaled score that moves only when the block's
            // maximum lies more than kPfSlack above it (see prefill_kernel); the four threads decide alike
            const float m_new = (rmax > m + kPfSlack) ? rmax : m;
            const float alpha = ex2_approx(m - m_new);
            const uint64_t c2x2 = pack_f32x2(c2, c2), mx2 = pack_f32x2(-m_new, -m_new);
            uint64_t lsum2 = 0;                           // two partial row sums, (+0, +0)
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                float a0, a1;
                unpack_f32x2(fma_f32x2(pack_f32x2(sv[i], sv[i + 1]), c2x2, mx2), a0, a1);
                const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                lsum2 = add_f32x2(lsum2, pack_f32x2(p0, p1));
                pk[i >> 1] = pack_bf16(p0, p1);
            }
            // this part of P(j) as bf16 pairs over the first 16 of the columns this thread read: the A operand
            // of O += P V (row = lane, two keys per column)
            tmem_st16u(tS, pk);
            {
                float s0, s1;
                unpack_f32x2(lsum2, s0, s1);
                l = l * alpha + (s0 + s1);                // this thread's part of the row sum
            }
            m = m_new;
            // rescale this thread's 32 columns of O where the reference moved (rare): only then must
            // O += P(j-1) V(j-1) have finished
            if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
                ok = mbar_wait(smem_u32(&bar_o[(j - 1) & 1]), ((j - 1) >> 1) & 1) && ok;
                tc_fence_after();
                float ov[32];
                tmem_ld32(t_lane + 256 + part * 32, ov);
#pragma unroll
                for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                tmem_st32(t_lane + 256 + part * 32, ov);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();                                 // one arrival per warp: hundreds of arrivals on one barrier word would queue up
            if (lane == 0) mbar_arrive(smem_u32(&bar_p[j & 1]));
        }
        ok = mbar_wait(smem_u32(&bar_o[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
    }
    tc_fence_after();
    const bool gave_up = !__syncthreads_and(ok);
    if (gave_up) {
        if (tid == 0) flag_error(p.hdr, 6 /* SPD_ERR_TIMEOUT */, -1);
    } else if (wid < 16) {
        // ---- the row sum is the four parts together; then each thread normalises its 32 channels into shared
        //      memory (Q and the first K slot are free: every MMA is done), and the warps store whole rows
        //      (16-byte chunks XOR-swizzled by the row against bank conflicts); rows past the prompt's end are
        //      not stored
        xch[part * 128 + row] = l;
        asm volatile("bar.sync %0, 128;" ::"r"(quad_bar) : "memory");
        const float inv = 1.f / ((xch[row] + xch[128 + row]) + (xch[256 + row] + xch[384 + row]));
        uint8_t *stage = base;
        const int rows_live = len - (qb * kPfBlock + quarter * 32);            // rows of this lane quarter that belong to the prompt
        const int64_t tok0 = static_cast<int64_t>(first) + qb * kPfBlock + quarter * 32;
        uint8_t *dst = reinterpret_cast<uint8_t *>(p.out);
        float ov[32];
        tmem_ld32(t_lane + 256 + part * 32, ov);
        if (p.out_bf16) {                                                     // 256-byte rows
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                *reinterpret_cast<uint4 *>(stage + row * 256 + (((part * 4 + q4) ^ (row & 7)) << 4)) =
                    make_uint4(pack_bf16(ov[8 * q4] * inv, ov[8 * q4 + 1] * inv), pack_bf16(ov[8 * q4 + 2] * inv, ov[8 * q4 + 3] * inv),
                               pack_bf16(ov[8 * q4 + 4] * inv, ov[8 * q4 + 5] * inv), pack_bf16(ov[8 * q4 + 6] * inv, ov[8 * q4 + 7] * inv));
            asm volatile("bar.sync %0, 128;" ::"r"(quad_bar) : "memory");
            // each of the four warps stores 8 of the quarter's 32 rows, two rows per instruction
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const int r = part * 8 + 2 * it + (lane >> 4), ch = lane & 15, rr = quarter * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 256 + ch * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 7)) << 4));
            }
        } else {                                                              // 512-byte rows
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4)
                *reinterpret_cast<float4 *>(stage + row * 512 + (((part * 8 + q4) ^ (row & 7)) << 4)) =
                    make_float4(ov[4 * q4] * inv, ov[4 * q4 + 1] * inv, ov[4 * q4 + 2] * inv, ov[4 * q4 + 3] * inv);
            asm volatile("bar.sync %0, 128;" ::"r"(quad_bar) : "memory");
            // each of the four warps stores 8 of the quarter's 32 rows, one row per instruction
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int r = part * 8 + it, rr = quarter * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 512 + lane * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 512 + ((lane ^ (rr & 7)) << 4));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPwTmemCols) : "memory");
}

}  // namespace spd
