// Prefill: causal self-attention over each user's prompt (protocol step 2; Fig. 3 step 0), and the
// hand-over of the prompt's K/V rows to the private paged cache that decode reads.
//
// This is the one dense contraction next to the decode path, so it runs on the fifth-generation
// tensor cores: tcgen05.mma with operands in 128-byte-swizzled shared memory (filled by TMA) or in
// tensor memory (TMEM), accumulators in TMEM.  One CTA owns 128 query rows of one (user, query head)
// and walks 64-key blocks up to the diagonal:
//     S = Q K^T            128 x 64 x head_dim    -> TMEM, two buffers: columns [0, 64) and [64, 128)
//     online softmax       one query row per thread (TMEM lane = row); P goes back into the first 32
//                          columns of S's own buffer as bf16 pairs
//     O += P V             128 x head_dim x 64    -> TMEM columns [128, 256); P is read from TMEM, V from
//                          shared memory
// Shared-memory bandwidth is what bounds this loop (every MMA streams its shared-memory operands again),
// which is why P never touches shared memory.
// Warp-specialised software pipeline: four warps do the softmax, one thread of a fifth warp issues every
// TMA load and the S products, one thread of a sixth the P V products.  S(j+1) is computed while the softmax warps work on S(j), and O takes block j
// in under the exponentials of block j+1.  They hand over through mbarriers only (S ready, P ready, O
// updated): no CTA-wide barrier inside the loop.  K and V blocks sit in two-slot rings with their own
// barriers; every wait is bounded and TMEM is freed on every way out.
// 96 KB of shared memory and 256 TMEM columns per CTA, so two CTAs share an SM and one's softmax runs
// under the other's MMAs.  bf16, head_dim 128.
#pragma once

#include "spd_kernels.cuh"

namespace spd {

constexpr int kPfBlock = 128;                       // query rows per CTA
constexpr int kPfKeys = 64;                         // keys per block
constexpr int kPfQBox = kPfBlock * 128;             // one swizzled box of Q or P: 128 rows x 128 bytes
constexpr int kPfQTile = 2 * kPfQBox;               // Q: 128 rows x 128 channels = two boxes
constexpr int kPfKvBox = kPfKeys * 128;             // one swizzled box of K or V: 64 rows x 128 bytes
constexpr int kPfKvTile = 2 * kPfKvBox;             // 64 keys x 128 channels = two boxes
constexpr int kPfTmemCols = 256;                    // S: 2 x 64, O: 128
constexpr float kPfSlack = 8.f;                     // log2 units the running reference may lag the maximum by

struct PrefillParams {
    int32_t B, Hq, Hkv;
    int64_t T;                   // tokens of all prompts together
    float sm_scale;
    const int32_t *tok_indptr;   // [B+1] token offsets of the users
    void *out;                   // [T][Hq][128]
    int32_t out_bf16;
    int32_t *hdr;
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

// Shared-memory matrix descriptor of the tensor core: start address, leading and stride byte offsets
// (all in 16-byte units), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = static_cast<uint64_t>((saddr >> 4) & 0x3FFFu);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B K-major or MN-major, M = 128, N = n.
__device__ __forceinline__ constexpr uint32_t umma_idesc(bool b_mn_major, uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
          "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
          "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
          "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}

// 64 consecutive fp32 columns of this thread's TMEM lane, one load and one wait.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64]) {
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]),
          "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
          "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
          "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
          "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr) : "memory");
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
// Two fp32 lanes per instruction on the FMA pipe (halves the issue slots of the softmax arithmetic).
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
// The same MMA with the A operand in TMEM (K-major: row = lane, two bf16 per column) and B in shared memory.
__device__ __forceinline__ void umma_bf16_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Which (user, query block) a CTA owns: blocks of `rows` query rows are numbered user by user, and within a
// user from the prompt's end backwards (the heaviest first).  Every warp works it out for itself: lane l sums
// the blocks of users [l C, (l + 1) C) (independent loads, no early exit), a prefix sum over the lanes finds the
// chunk that holds block `blk`, and that lane walks its chunk once more (cache hits now).  A user whose offsets
// are inconsistent ends the list: blocks of earlier users are served, nothing from there on.  qb < 0: no block.
__device__ __forceinline__ void prefill_find_block(const PrefillParams &p, int rows, int blk, int lane, int &qb, int &first, int &len) {
    qb = -1; first = 0; len = 0;
    const int C = (p.B + 31) / 32;
    const int u0 = lane * C, u1 = min(p.B, u0 + C);
    int sum = 0;
    bool bad = false;
#pragma unroll 4
    for (int u = u0; u < u1; ++u) {
        const int64_t a = p.tok_indptr[u], b = p.tok_indptr[u + 1];
        bad = bad || a < 0 || b < a || b > p.T;
        if (!bad) sum += static_cast<int>((b - a + rows - 1) / rows);
    }
    int inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += up;
    }
    const unsigned badmask = __ballot_sync(0xffffffffu, bad), hit = __ballot_sync(0xffffffffu, blk < inc);
    if (!hit) return;
    const int src = __ffs(hit) - 1;
    if (badmask & ((1u << src) - 1u)) return;          // an inconsistent user in an earlier chunk
    int r_qb = -1, r_first = 0, r_len = 0;
    if (lane == src) {
        int rem = blk - (inc - sum);
        for (int u = u0; u < u1; ++u) {
            const int64_t a = p.tok_indptr[u], b = p.tok_indptr[u + 1];
            if (a < 0 || b < a || b > p.T) break;     // the sum stopped here too, so rem was used up before
            const int nb = static_cast<int>((b - a + rows - 1) / rows);
            if (rem < nb) { r_qb = nb - 1 - rem; r_first = static_cast<int>(a); r_len = static_cast<int>(b - a); break; }
            rem -= nb;
        }
    }
    qb = __shfl_sync(0xffffffffu, r_qb, src);
    first = __shfl_sync(0xffffffffu, r_first, src);
    len = __shfl_sync(0xffffffffu, r_len, src);
}

// Q, K x2, V x2, then eleven mbarriers and one word; the kernel has no static shared memory, so the
// 1024-byte alignment of the tiles costs nothing and two CTAs fit one SM.
constexpr size_t prefill_smem_bytes() { return kPfQTile + 4 * static_cast<size_t>(kPfKvTile) + 128; }   // 11 x 8 + 4 <= 128

constexpr int kPfThreads = 192;   // 4 softmax warps + 2 warps with one issuing thread each

__global__ void __launch_bounds__(kPfThreads, 2)
prefill_kernel(const __grid_constant__ PrefillParams p, const __grid_constant__ CUtensorMap mq,
               const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv) {
    extern __shared__ __align__(1024) uint8_t base[];
    const uint32_t Qs = smem_u32(base), Ks = Qs + kPfQTile, Vs = Ks + 2 * kPfKvTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + kPfQTile + 4 * kPfKvTile);
    uint64_t &bar_q = bars[0];                                             // Q loaded
    uint64_t *bar_o = bars + 1;                                            // O has taken in the block whose P was in S buffer 0 / 1
    uint64_t *bar_p = bars + 3;                                            // P written into S buffer 0 / 1
    uint64_t *bar_k = bars + 5, *bar_v = bars + 7, *bar_s = bars + 9;     // K / V slot loaded; S buffer ready
    uint32_t &tmem_slot = *reinterpret_cast<uint32_t *>(bars + 11);
    const int tid = threadIdx.x, wid = tid >> 5;
    const int h = blockIdx.y, kvh = h / (p.Hq / p.Hkv);

    if (tid == 128) { prefetch_tensormap(&mq); prefetch_tensormap(&mk); prefetch_tensormap(&mv); }   // needed right after the search below
    int qb, first, len;
    prefill_find_block(p, kPfBlock, blockIdx.x, tid & 31, qb, first, len);
    if (qb < 0) return;   // uniform over the CTA: no barrier, no TMEM touched yet
    const int nkv = 2 * (qb + 1);   // 64-key blocks up to and including the diagonal

    // K and V of key block j live in slot j & 1 of their rings; K is free again once S(j) exists, V once
    // O has taken block j in.
    auto load_k = [&](int j) {
        const uint32_t bar = smem_u32(&bar_k[j & 1]);
        mbar_expect_tx(bar, kPfKvTile);
        tma_load_3d(Ks + (j & 1) * kPfKvTile, &mk, 0, kvh, first + j * kPfKeys, bar);
        tma_load_3d(Ks + (j & 1) * kPfKvTile + kPfKvBox, &mk, 64, kvh, first + j * kPfKeys, bar);
    };
    auto load_v = [&](int j) {
        const uint32_t bar = smem_u32(&bar_v[j & 1]);
        mbar_expect_tx(bar, kPfKvTile);
        tma_load_3d(Vs + (j & 1) * kPfKvTile, &mv, 0, kvh, first + j * kPfKeys, bar);
        tma_load_3d(Vs + (j & 1) * kPfKvTile + kPfKvBox, &mv, 64, kvh, first + j * kPfKeys, bar);
    };
    if (tid == 128) {     // the issuing thread sets the barriers up and starts the first loads before anything else happens
        for (int b = 0; b < 11; ++b) mbar_init(smem_u32(&bars[b]), (b == 3 || b == 4) ? 4 : 1);   // P written: every softmax thread arrives
        fence_mbar_init();
        fence_proxy_async();
        const uint32_t bq = smem_u32(&bar_q);
        mbar_expect_tx(bq, kPfQTile);
        tma_load_3d(Qs, &mq, 0, h, first + qb * kPfBlock, bq);
        tma_load_3d(Qs + kPfQBox, &mq, 64, h, first + qb * kPfBlock, bq);
        load_k(0);
        load_v(0);
        load_k(1);            // nkv >= 2 always: a query block spans two key blocks on the diagonal
        load_v(1);
    }
    if (wid == 0) {       // one warp allocates the accumulator columns for the CTA
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kPfTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(wid * 32) << 16);   // this warp's 32 lanes
    const uint32_t tO = tmem + 2 * kPfKeys;     // S buffers at columns [0, 64) and [64, 128), O at [128, 256)

    auto mma_s = [&](int j) {                    // S(j) = Q K(j)^T into S buffer j & 1; 16 channels per MMA
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint64_t a = umma_desc(Qs + (kk >> 2) * kPfQBox + (kk & 3) * 32, 16, 1024);
            const uint64_t b = umma_desc(Ks + (j & 1) * kPfKvTile + (kk >> 2) * kPfKvBox + (kk & 3) * 32, 16, 1024);
            umma_bf16(tmem + (j & 1) * kPfKeys, a, b, umma_idesc(false, kPfKeys), kk > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bar_s[j & 1]));
    };
    const float c2 = p.sm_scale * kLog2e;   // scores in log2 units
    const int row = tid;                     // query row of a softmax thread within the block
    float l = 0.f;
    // Every wait is bounded.  A wait that runs out clears `ok` and the thread carries on (with garbage, but
    // towards the same end): nothing in the loop waits for all threads, so nobody can be left behind.
    bool ok = true;

    // One thread cannot issue MMAs faster than about one per hundred cycles, whatever their size, while the
    // tensor core takes them from two threads at nearly twice that rate: so two threads issue, one the
    // S = Q K^T products (and the TMA loads), the other the O += P V products.  MMAs of different threads are
    // not ordered by issue, so where one's operands or accumulator depend on the other's work it waits for the
    // commit barrier, never for the issue.  All barriers that a thread may find two phases ahead exist twice
    // (per S buffer), so that parity never aliases.
    if (wid == 4) {
        // ---------------- first issuing thread: TMA loads and S = Q K^T -------------------------------------
        if (tid == 128) {
            ok = mbar_wait(smem_u32(&bar_q), 0) && mbar_wait(smem_u32(&bar_k[0]), 0);
            mma_s(0);
            for (int j = 0; j < nkv; ++j) {
                if (j + 1 < nkv) {
                    ok = mbar_wait(smem_u32(&bar_k[(j + 1) & 1]), ((j + 1) >> 1) & 1) && ok;
                    // S(j+1) goes where S(j-1) and then P(j-1) were, and V(j+1) where V(j-1) was: both are free
                    // once O has taken block j-1 in
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
    } else if (wid == 5) {
        // ---------------- second issuing thread: O += P V -----------------------------------------------------
        if (tid == 160) {
            for (int j = 0; j < nkv; ++j) {
                ok = mbar_wait(smem_u32(&bar_p[j & 1]), (j >> 1) & 1) && ok;       // P(j) is written and O rescaled
                ok = mbar_wait(smem_u32(&bar_v[j & 1]), (j >> 1) & 1) && ok;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {       // 16 keys per MMA; P comes from TMEM (8 columns per 16 keys)
                    // V is [key][channel]: MN-major for the B operand; 8-key groups 1024 bytes apart, 64-channel boxes one box apart
                    const uint64_t b = umma_desc(Vs + (j & 1) * kPfKvTile + kk * 2048, kPfKvBox, 1024);
                    umma_bf16_ta(tO, tmem + (j & 1) * kPfKeys + kk * 8, b, umma_idesc(true, 128), (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_o[j & 1]));
            }
            ok = mbar_wait(smem_u32(&bar_o[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
        }
    } else {
        // ---------------- softmax warps: one query row per thread -------------------------------------------
        float m = -INFINITY;
        for (int j = 0; j < nkv; ++j) {
            ok = mbar_wait(smem_u32(&bar_s[j & 1]), (j >> 1) & 1) && ok;           // S(j) is there
            tc_fence_after();
            float sv[64];
            tmem_ld64(t_lane + (j & 1) * kPfKeys, sv);
            // key (64 j + col) is visible to row (128 qb + row) iff it does not lie ahead of it; only the two
            // blocks on the diagonal hide anything; `ahead` = first column of this block hidden from this row
            if (j >= 2 * qb) {
                const int ahead = (kPfBlock * qb + row) - kPfKeys * j + 1;
#pragma unroll
                for (int i = 0; i < 64; ++i) sv[i] = (i >= ahead) ? -INFINITY : sv[i];
            }
            // m is kept in log2 units of the scaled score; the maximum is taken on the raw scores (the scale
            // is positive) and the scale rides on the fused multiply-add that feeds ex2.  m is a reference
            // point, not necessarily the exact maximum: it moves only when the block's maximum lies more than
            // kPfSlack above it, so weights reach 2^kPfSlack at most (harmless in fp32 and bf16, and O and l
            // carry the same factor, which the final division removes) and O is seldom rescaled.
            float r4[4];                                 // four chains of three-input maxima
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                r4[c] = fmax3(sv[16 * c], sv[16 * c + 1], sv[16 * c + 2]);
#pragma unroll
                for (int i = 3; i < 15; i += 2) r4[c] = fmax3(r4[c], sv[16 * c + i], sv[16 * c + i + 1]);
                r4[c] = fmaxf(r4[c], sv[16 * c + 15]);
            }
            const float rmax = fmaxf(fmax3(r4[0], r4[1], r4[2]), r4[3]) * c2;   // finite from the first block on: key 0 is visible to every row
            const float m_new = (rmax > m + kPfSlack) ? rmax : m;
            const float alpha = ex2_approx(m - m_new);
            uint32_t pk[32];
            float lsum = 0.f;
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
                lsum = s0 + s1;
            }
            l = l * alpha + lsum;
            m = m_new;
            // rescale O where the reference moved (rare): only then must O += P(j-1) V(j-1) have finished
            if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
                ok = mbar_wait(smem_u32(&bar_o[(j - 1) & 1]), ((j - 1) >> 1) & 1) && ok;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float ov[32];
                    tmem_ld32(t_lane + (tO - tmem) + c * 32, ov);
#pragma unroll
                    for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                    tmem_st32(t_lane + (tO - tmem) + c * 32, ov);
                }
            }
            // P(j) as bf16 pairs over the first 32 columns of S(j)'s buffer: the A operand of O += P V, read
            // by the tensor core straight from TMEM (row = lane, two keys per column)
            tmem_st32u(t_lane + (j & 1) * kPfKeys, pk);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();                                 // one arrival per warp: arrivals on one barrier word queue up
            if ((tid & 31) == 0) mbar_arrive(smem_u32(&bar_p[j & 1]));
        }
        ok = mbar_wait(smem_u32(&bar_o[(nkv - 1) & 1]), ((nkv - 1) >> 1) & 1) && ok;
    }
    tc_fence_after();
    const bool gave_up = !__syncthreads_and(ok);
    if (gave_up) {
        if (tid == 0) flag_error(p.hdr, 6 /* SPD_ERR_TIMEOUT */, -1);
    } else if (wid < 4) {
        // ---- normalise this thread's row into shared memory (the Q and K tiles are free by now), then each
        //      warp stores its own 32 rows with whole rows per instruction; 16-byte chunks are XOR-swizzled
        //      by the row so that neither side meets bank conflicts; rows past the prompt's end are not stored
        const float inv = 1.f / l;
        const int lane = tid & 31;
        uint8_t *stage = base;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            float ov[32];
            tmem_ld32(t_lane + (tO - tmem) + c * 32, ov);
            if (p.out_bf16) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<uint4 *>(stage + row * 256 + (((c * 4 + q4) ^ (row & 7)) << 4)) =
                        make_uint4(pack_bf16(ov[8 * q4] * inv, ov[8 * q4 + 1] * inv), pack_bf16(ov[8 * q4 + 2] * inv, ov[8 * q4 + 3] * inv),
                                   pack_bf16(ov[8 * q4 + 4] * inv, ov[8 * q4 + 5] * inv), pack_bf16(ov[8 * q4 + 6] * inv, ov[8 * q4 + 7] * inv));
            } else {
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4)
                    *reinterpret_cast<float4 *>(stage + row * 512 + (((c * 8 + q4) ^ (row & 7)) << 4)) =
                        make_float4(ov[4 * q4] * inv, ov[4 * q4 + 1] * inv, ov[4 * q4 + 2] * inv, ov[4 * q4 + 3] * inv);
            }
        }
        __syncwarp();
        const int rows_live = len - (qb * kPfBlock + wid * 32);            // rows of this warp that belong to the prompt
        const int64_t tok0 = static_cast<int64_t>(first) + qb * kPfBlock + wid * 32;
        if (p.out_bf16) {
            uint8_t *dst = reinterpret_cast<uint8_t *>(p.out);
#pragma unroll 4
            for (int it = 0; it < 16; ++it) {
                const int r = 2 * it + (lane >> 4), ch = lane & 15, rr = wid * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 256 + ch * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 7)) << 4));
            }
        } else {
            uint8_t *dst = reinterpret_cast<uint8_t *>(p.out);
#pragma unroll 4
            for (int r = 0; r < 32; ++r) {
                const int rr = wid * 32 + r;
                if (r < rows_live)
                    *reinterpret_cast<uint4 *>(dst + ((tok0 + r) * p.Hq + h) * 512 + lane * 16) =
                        *reinterpret_cast<const uint4 *>(stage + rr * 512 + ((lane ^ (rr & 7)) << 4));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPfTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------------
// The prompt's K and V rows into the private paged cache (what prefill leaves for decode): one CTA
// per token.  Token t of user u goes to page indices[page_indptr[u] + t / 16], slot t % 16.  A user
// whose listed pages cannot hold its prompt is flagged and skipped; seq_lens[u] is set for the rest.
struct PromptKvParams {
    int32_t B, Hkv, row_bytes;
    int64_t T;
    const uint8_t *k, *v;            // [T][Hkv][row_bytes]
    const int32_t *tok_indptr;
    uint8_t *k_pool, *v_pool;
    int32_t num_pages;
    const int32_t *page_indptr, *page_indices;
    int32_t *lens;
    int32_t *hdr;
};

__global__ void __launch_bounds__(128) prompt_kv_kernel(PromptKvParams p) {
    __shared__ int64_t dst_row;
    const int64_t tok = blockIdx.x;
    if (tok == p.T) {                              // the extra block: users without a prompt hold no tokens
        for (int u = threadIdx.x; u < p.B; u += blockDim.x)
            if (p.tok_indptr[u + 1] == p.tok_indptr[u]) p.lens[u] = 0;
        return;
    }
    if (threadIdx.x == 0) {
        int64_t off = -1;
        int lo = 0, hi = p.B;                      // user u with tok_indptr[u] <= tok < tok_indptr[u + 1]
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (p.tok_indptr[mid] <= tok) lo = mid; else hi = mid; }
        while (lo + 1 < p.B && p.tok_indptr[lo + 1] <= tok) ++lo;       // skip users without tokens
        const int u = lo;
        const int64_t a = p.tok_indptr[u], b = p.tok_indptr[u + 1], t = tok - a;
        const int64_t plo = p.page_indptr[u], phi = p.page_indptr[u + 1];
        bool good = a <= tok && tok < b && plo >= 0 && phi >= plo && phi <= p.page_indptr[p.B] &&
                    (b - a) <= (phi - plo) * kPage && p.page_indices != nullptr;
        if (good) {
            const int64_t page = p.page_indices[plo + t / kPage];
            if (page >= 0 && page < p.num_pages) off = ((page * p.Hkv) * kPage + t % kPage) * p.row_bytes;
            else good = false;
        }
        if (!good) flag_error(p.hdr, 4 /* SPD_ERR_BAD_PAGE */, u);
        else if (t == 0) p.lens[u] = static_cast<int32_t>(b - a);
        dst_row = off;
    }
    __syncthreads();
    const int64_t off = dst_row;
    if (off < 0) return;
    const int chunks = p.row_bytes / 16, total = p.Hkv * chunks;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int hh = i / chunks, c = i - hh * chunks;
        const int64_t src = (tok * p.Hkv + hh) * p.row_bytes + c * 16;
        const int64_t dst = off + static_cast<int64_t>(hh) * kPage * p.row_bytes + c * 16;
        *reinterpret_cast<uint4 *>(p.k_pool + dst) = *reinterpret_cast<const uint4 *>(p.k + src);
        *reinterpret_cast<uint4 *>(p.v_pool + dst) = *reinterpret_cast<const uint4 *>(p.v + src);
    }
}

}  // namespace spd
