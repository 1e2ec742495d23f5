// Device-side building blocks for the partitioned decode-attention kernels (sm_100a):
// mbarrier + TMA tile loads, ldmatrix / mma.sync wrappers, and the parameter blocks that the
// host fills.  Everything here is specific to this library; nothing is shared with the CPU oracle.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spd {

constexpr int kPage = 16;             // tokens per KV page
constexpr int kHeadsPerItem = 8;      // query heads one warp carries for one KV head
constexpr int kMinTilesPerWarp = 4;   // default: do not spread tiny batches thinner than this (tiles per share)
constexpr int kMaxGrid = 256;         // CTAs (one per SM) the share tables are sized for
constexpr int kMaxWarpsPerCta = 16;
constexpr uint32_t kWaitLimit = 1u << 22;  // bounded mbarrier polling (each poll may block ~us)

// Words of the workspace header (int32 each).
enum HdrWord {
    HDR_STATUS = 0,        // 0 or an spd_status code, sticky
    HDR_BAD_ENC = 1,       // 0 = none, else 0x7fffffff - lowest flagged user (atomicMax)
    HDR_BATCH = 2,         // batch size of the last call (size of the per-user flag array)
    HDR_NSEQ = 3,          // sequences of the last call (size of the ticket array)
    HDR_SM_LAUNCHES = 4,   // attention launches that compared their CTAs' SMs with the previous launch's
    HDR_SM_MOVES = 5,      // CTAs of those launches that found themselves on another SM than last time
    HDR_GRID_EXITS = 6,    // CTAs of the running launch that have finished (only counted by launches that append); zero between calls
    HDR_WORDS = 64
};

// The plan of the last planning launch, kept in the workspace (int32 words): what a later launch with the same
// lengths loads instead of deriving it again, and what the debugging export reads.
enum PlanWord {
    PLAN_TAG = 0,          // id (epoch) of the launch that wrote the plan; 0 = none
    PLAN_T = 1,            // tiles in the stream
    PLAN_A = 2,            // warps that own a share
    PLAN_GRID = 3,         // CTAs of the grid the plan was cut for
    PLAN_WARPS = 4,        // warps per CTA
    PLAN_B = 5,            // users
    PLAN_S = 6,            // sequences per user
    PLAN_PARTS = 7,        // which partitions the call read (bit 0 private, bit 1 public)
    PLAN_HDR_WORDS = 16,
    PLAN_WQ = PLAN_HDR_WORDS,                 // [kMaxGrid] share weight of each CTA
    PLAN_SMID = PLAN_WQ + kMaxGrid,           // [kMaxGrid] 1 + SM the CTA ran on at the last launch (0 = unknown)
    PLAN_BND = PLAN_SMID + kMaxGrid,          // [kMaxGrid * kMaxWarpsPerCta + 1] share boundaries
    PLAN_REC = PLAN_BND + kMaxGrid * kMaxWarpsPerCta + 16,   // [kMaxGrid * kMaxWarpsPerCta][8] where each warp starts
    PLAN_WORDS = PLAN_REC + kMaxGrid * kMaxWarpsPerCta * 8
};

// One KV partition as the kernels see it.
struct PartDev {
    const int32_t *indptr;
    const int32_t *indices;
    const int32_t *lens;
    int32_t num_pages;
    int32_t present;
};

enum OutMode { OUT_PARTIAL = 0, OUT_FINAL = 1 };
// How a launch gets its plan: derives it and keeps only the boundaries for inspection; derives it and stores all of
// it for later launches; or loads what an earlier launch on this workspace stored (same lengths, same grid).
enum PlanMode { PLAN_DERIVE = 0, PLAN_DERIVE_STORE = 1, PLAN_LOAD = 2 };

struct Params {
    int32_t B, Hq, Hkv, g;
    int32_t hgroups;        // head groups per KV head: max(1, g / 8)
    int32_t geff;           // query heads per item: min(g, 8)
    int32_t S;              // sequences per user = Hkv * hgroups
    int32_t num_warps;      // warps in the attention grid
    float sm_scale;
    const void *q;
    PartDev part[2];        // 0 = private, 1 = public
    // workspace
    int32_t *hdr;
    int32_t *bad;           // [B] per-user flags: holds `epoch` if the user was flagged by this call
    int32_t *tickets;       // [B * S] pieces delivered so far per sequence; zero between calls
    int32_t epoch;          // non-zero id of this call
    float2 *rates;          // [3][kMaxGrid] per-CTA (share weight, cycles) of earlier launches
    int32_t rate_sel;       // attention launches on this workspace so far: this launch writes third rate_sel % 3,
                            // reads (rate_sel + 1) % 3
    int32_t *plan;          // [PLAN_WORDS] the stored plan
    int32_t plan_mode;      // PlanMode
    int32_t plan_early;     // PLAN_LOAD: the plan may be read before the previous kernel on the stream has finished
    int32_t plan_tag;       // what PLAN_TAG must hold for a plan to be loaded / holds once this launch has stored one
    int32_t min_tiles;      // fewest tiles a share may hold (>= 1)
    int32_t uniform;        // non-zero: equal shares, the rate table is ignored
    float *scratch;         // [2 * num_warps][8 * D + 16]
    // outputs
    int32_t mode;           // OutMode
    float *po, *pm, *pl;    // OUT_PARTIAL destination
    const float *in_o, *in_m, *in_l;  // OUT_FINAL: optional partial to merge in (may be null)
    void *out;              // OUT_FINAL destination
    int32_t out_bf16;
    // optional append inside the launch (protocol step 3a): the new token's K and V rows, [B][Hkv][D] in the pools'
    // dtype, go to position lens[u] of the public partition, which the launch reads as one token longer; the last
    // CTA to finish adds one to the length of every user that was not flagged.  k_new == nullptr: no append.
    const uint8_t *k_new, *v_new;
    uint8_t *k_pool_w, *v_pool_w;   // the public pools, writable
    int32_t *lens_w;                // the public seq_lens, writable
    // optional monitor: softmax mass on tokens [watch_lo[u], watch_hi[u]) of the private partition
    const int32_t *watch_lo, *watch_hi;   // [B]
    float *watch_out;                      // [B][Hq]; null = not watching
};

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the polling limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// L2 policy for data that is read once: first in line to be evicted.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// One 2-D TMA tile load (no multicast): box at (x, y) of the tensor map into shared memory.  KV tiles
// are read once per call, so they carry the evict-first hint (measured: 2-3 % faster than without).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}

// Brings a tensor map (a kernel parameter) into the descriptor cache ahead of its first use.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Programmatic dependent launch: let the next kernel on the stream start its own read-only preamble
// early, and wait until the previous kernel on the stream has completed and its writes are visible.
// Both are no-ops when the launch did not ask for programmatic serialisation.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Raise the sticky status and remember the lowest flagged user.
__device__ __forceinline__ void flag_error(int32_t *hdr, int code, int user) {
    atomicCAS(&hdr[HDR_STATUS], 0, code);
    if (user >= 0) atomicMax(&hdr[HDR_BAD_ENC], 0x7fffffff - user);
}

}  // namespace spd
