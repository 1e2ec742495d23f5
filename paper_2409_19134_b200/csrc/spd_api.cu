// Host side of libspd.so: argument checks, workspace layout, TMA descriptors, kernel launches.
// The C ABI is declared in include/spd.h.
#include "spd.h"

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "spd_kernels.cuh"
#include "spd_prefill.cuh"
#include "spd_prefill_pair.cuh"
#include "spd_prefill_fma.cuh"

namespace {

using namespace spd;

std::atomic<int64_t> g_launches{0};

// Optional timing of the three kernels of a call with CUDA events on the caller's stream.
struct Profiler {
    std::mutex mu;
    bool on = false;
    int jobs = 0, cap = 0;
    std::vector<cudaEvent_t> ev;   // 2 per call: before and after the kernel
} g_prof;

void prof_mark(int job, int k, cudaStream_t st) {
    if (job >= 0) cudaEventRecord(g_prof.ev[2 * job + k], st);
}

std::atomic<uint32_t> g_epoch{0};
std::atomic<int> g_bf16_math{0};   // 0 = tensor cores (default), 1 = FMA pipes (comparison arm)
std::atomic<int> g_prefill_rows{0};   // query rows per prefill CTA: 0 = by mean prompt length, 128, 256
std::atomic<int> g_min_tiles{kMinTilesPerWarp};   // fewest page tiles a share of the tile stream may hold
std::atomic<int> g_uniform_shares{0};             // 1 = equal shares, the measured rates are ignored
std::atomic<int> g_pdl{-1};                       // programmatic launch: -1 = not decided yet (environment), 0 off, 1 on

// What the host remembers about a workspace (keyed by its address): the attention launches made on it so far, and
// at which of them each kind of call last stored its plan.  The kernel rotates through the three thirds of the
// workspace's rate table by the launch count, so it must advance by exactly one per attention launch on that
// workspace whatever else the process launches in between.
struct WsHostState {
    uint64_t launches = 0;
    uint64_t stored_at[3] = {~0ull, ~0ull, ~0ull};
};

// Registers one attention launch.  *early_plan: a launch that loads a stored plan may read it before the
// previous kernel on the stream has finished when that kernel is not the one that stored it (the launch before
// the previous one has left every SM by the time this one starts, since each CTA takes a whole SM).
uint32_t register_launch(const void *ws, int slot, int plan_mode, bool *early_plan) {
    static std::mutex mu;
    static std::unordered_map<const void *, WsHostState> table;
    std::lock_guard<std::mutex> lock(mu);
    WsHostState &st = table[ws];
    const uint64_t n = st.launches++;
    *early_plan = plan_mode == PLAN_LOAD && st.stored_at[slot] != ~0ull && n >= st.stored_at[slot] + 2;
    if (plan_mode == PLAN_DERIVE_STORE) st.stored_at[slot] = n;
    if (plan_mode == PLAN_DERIVE) st.stored_at[slot] = ~0ull;
    return static_cast<uint32_t>(n % 3u);
}

bool programmatic_launch() {
    int v = g_pdl.load();
    if (v < 0) {
        v = getenv("SPD_NO_PDL") == nullptr ? 1 : 0;
        g_pdl.store(v);
    }
    return v != 0;
}
constexpr int64_t kPrefillPairFrom = 768;    // mean prompt length from which the 256-row kernel is used

// Ids of calls: non-zero, so that a zeroed workspace matches none.
int32_t next_epoch() {
    uint32_t e = ++g_epoch;
    if ((e & 0x7fffffffu) == 0) e = ++g_epoch;
    return static_cast<int32_t>(e & 0x7fffffffu);
}

struct DeviceInfo {
    int sms = 0;
    bool ok = false;
};

// Per-device facts, looked up once.
spd_status device_info(DeviceInfo *out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPD_ERR_CUDA;
    // The tensor maps are encoded through the driver API, which wants the device's context current on the CALLING
    // thread; the runtime only makes it so at a thread's first call that needs a context.  A host thread that has
    // made no such call yet (a worker that only ever calls this library) gets it here, once: a stream query does it
    // and neither allocates nor waits.
    static thread_local int bound_dev = -1;
    if (bound_dev != dev) {
        const cudaError_t e = cudaStreamQuery(cudaStreamLegacy);
        if (e != cudaSuccess && e != cudaErrorNotReady) return SPD_ERR_CUDA;
        bound_dev = dev;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev].ok) {
        int sms = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SPD_ERR_CUDA;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SPD_ERR_CUDA;
        if (major != 10) return SPD_ERR_UNSUPPORTED;   // built for sm_100a only
        cache[dev].sms = sms;
        cache[dev].ok = true;
    }
    *out = cache[dev];
    return SPD_OK;
}

// A copy stream and two events per host thread and device for the host-buffer entry point, made at the thread's
// first large call on the device and kept (no device memory is involved).
constexpr int kHostStepParts = 2;     // a large batch is served in this many parts (8 status words each: at most 8); four measured no faster than two
struct HostStepStreams {
    cudaStream_t copy = nullptr;
    cudaEvent_t q_up[kHostStepParts] = {}, done[kHostStepParts] = {};   // part i's q is on the device; part i's kernel has finished
};

spd_status host_step_streams(HostStepStreams *out) {
    static thread_local HostStepStreams cache[64];     // per host thread: two threads may serve two batches at once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPD_ERR_CUDA;
    HostStepStreams &h = cache[dev];
    if (!h.copy) {
        HostStepStreams n;
        if (cudaStreamCreateWithFlags(&n.copy, cudaStreamNonBlocking) != cudaSuccess) return SPD_ERR_CUDA;
        for (int i = 0; i < kHostStepParts; ++i)
            if (cudaEventCreateWithFlags(&n.q_up[i], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&n.done[i], cudaEventDisableTiming) != cudaSuccess)
                return SPD_ERR_CUDA;
        h = n;
    }
    *out = h;
    return SPD_OK;
}

#ifndef SPD_TMA_L2_PROMOTION
#define SPD_TMA_L2_PROMOTION CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

constexpr size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace layout.  The header, the per-user flags and the tickets come first so that the status
// query can find them without knowing the shape.
struct WsLayout {
    size_t hdr, rates, plan, bad, tickets, scratch, partial_o, partial_m, partial_l, total;
};

// The part of the layout that the status query must find from the header alone: it depends only on the batch
// size and the number of sequences, which the kernels leave in the header.
struct WsHead {
    size_t hdr, rates, plan, bad, tickets, end;
};

constexpr size_t kPlanBytes = static_cast<size_t>(PLAN_WORDS) * 4;   // one stored plan
constexpr int kPlanSlots = 3;                                        // private only, public only, both partitions

WsHead ws_head(size_t batch, size_t seqs) {
    WsHead H;
    size_t off = 0;
    H.hdr = off;       off = align_up(off + HDR_WORDS * 4, 256);
    H.rates = off;     off = align_up(off + 3 * kMaxGrid * sizeof(float2), 256);
    H.plan = off;      off = align_up(off + kPlanSlots * kPlanBytes, 256);
    H.bad = off;       off = align_up(off + batch * 4, 256);
    H.tickets = off;   off = align_up(off + seqs * 4, 256);
    H.end = off;
    return H;
}

WsLayout ws_layout(const spd_shape &s, int sms) {
    WsLayout L;
    const size_t B = s.batch;
    const int g = s.num_q_heads / s.num_kv_heads;
    const size_t seqs = B * s.num_kv_heads * (g > kHeadsPerItem ? g / kHeadsPerItem : 1);
    const WsHead H = ws_head(B, seqs);
    L.hdr = H.hdr; L.rates = H.rates; L.plan = H.plan; L.bad = H.bad; L.tickets = H.tickets;
    size_t off = H.end;
    constexpr int wmax = MathBF16<128>::kWarps > MathF32<128, 1>::kWarps ? MathBF16<128>::kWarps : MathF32<128, 1>::kWarps;
    const size_t max_warps = static_cast<size_t>(sms) * wmax;
    L.scratch = off;   off = align_up(off + 2 * max_warps * slot_floats(s.head_dim) * 4, 256);
    const size_t rows = B * s.num_q_heads;
    L.partial_o = off; off = align_up(off + rows * s.head_dim * 4, 256);
    L.partial_m = off; off = align_up(off + rows * 4, 256);
    L.partial_l = off; off = align_up(off + rows * 4, 256);
    L.total = off;
    return L;
}

spd_status check_shape(const spd_shape *s) {
    if (!s) return SPD_ERR_INVALID_ARG;
    if (s->batch <= 0 || s->num_q_heads <= 0 || s->num_kv_heads <= 0) return SPD_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128) return SPD_ERR_UNSUPPORTED;
    if (s->page_size != kPage) return SPD_ERR_UNSUPPORTED;
    if (s->dtype != SPD_F32 && s->dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    if (s->num_q_heads % s->num_kv_heads != 0) return SPD_ERR_UNSUPPORTED;
    const int g = s->num_q_heads / s->num_kv_heads;
    if (!(g == 1 || g == 2 || g == 4 || g % 8 == 0)) return SPD_ERR_UNSUPPORTED;
    if (!(s->sm_scale == s->sm_scale)) return SPD_ERR_INVALID_ARG;
    return SPD_OK;
}

bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

spd_status check_kv(const spd_shape *s, const spd_paged_kv *kv) {
    if (!kv) return SPD_ERR_INVALID_ARG;
    if (kv->num_pages < 0) return SPD_ERR_INVALID_ARG;
    if (!kv->page_indptr || !kv->seq_lens) return SPD_ERR_INVALID_ARG;
    // page_indices may be null when no user lists a page (the device checks that before any read)
    if (kv->num_pages > 0 && (!kv->k_pool || !kv->v_pool)) return SPD_ERR_INVALID_ARG;
    if (misaligned(kv->k_pool, 128) || misaligned(kv->v_pool, 128)) return SPD_ERR_INVALID_ARG;
    // TMA row coordinates are 32-bit
    if (static_cast<int64_t>(kv->num_pages) * s->num_kv_heads * kPage >= (1ll << 31)) return SPD_ERR_UNSUPPORTED;
    return SPD_OK;
}

spd_status make_map(CUtensorMap *map, const spd_shape &s, const void *pool, int64_t num_pages) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SPD_ERR_CUDA;
    const bool bf = s.dtype == SPD_BF16;
    const cuuint64_t es = bf ? 2 : 4;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(s.head_dim),
                          static_cast<cuuint64_t>(num_pages) * s.num_kv_heads * kPage};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(s.head_dim) * es};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(bf ? 64 : s.head_dim), static_cast<cuuint32_t>(kPage)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                    const_cast<void *>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    bf ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, SPD_TMA_L2_PROMOTION,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) fprintf(stderr, "libspd: cuTensorMapEncodeTiled failed with CUresult %d\n", static_cast<int>(r));
    return r == CUDA_SUCCESS ? SPD_OK : SPD_ERR_CUDA;
}

template <class Math>
spd_status launch_attn(const Params &p_in, const CUtensorMap *maps, int sms, cudaStream_t st, bool pdl) {
    if (sms > kMaxGrid) return SPD_ERR_UNSUPPORTED;
    Params p = p_in;
    p.num_warps = sms * Math::kWarps;   // the plan cuts the tile stream into one share per warp of THIS grid
    // At least 117 KB, so that an SM never holds two of these CTAs whatever the variant needs: the kernel's
    // reasoning about which launch can still be running when the next but one starts rests on one CTA per SM.
    const size_t smem = attn_smem_bytes<Math>(sms) > 117 * 1024 ? attn_smem_bytes<Math>(sms) : 117 * 1024;
    static std::once_flag once[64];
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t attr_err = cudaSuccess;
    std::call_once(once[dev & 63], [&] {
        attr_err = cudaFuncSetAttribute(attn_kernel<Math>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem));
    });
    if (attr_err != cudaSuccess) {
        fprintf(stderr, "libspd: cudaFuncSetAttribute(dynamic shared memory %zu): %s\n", smem, cudaGetErrorString(attr_err));
        return SPD_ERR_CUDA;
    }
    // Programmatic stream serialisation (pdl): this kernel's read-only preamble may overlap the tail of the
    // previous kernel on the stream if that kernel allows it (the attention kernel does).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms);
    cfg.blockDim = dim3(Math::kWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, attn_kernel<Math>, p, maps[0], maps[1], maps[2], maps[3]);
    ++g_launches;
    if (err != cudaSuccess) fprintf(stderr, "libspd: launch of the attention kernel: %s\n", cudaGetErrorString(err));
    return err == cudaSuccess ? SPD_OK : SPD_ERR_CUDA;
}

// What one library call boils down to: one launch of the attention kernel.
struct Job {
    const spd_shape *shape;
    const void *q;
    const spd_paged_kv *part[2];   // private, public; either may be null (absent)
    int mode;
    spd_partial pout;              // OUT_PARTIAL
    const spd_partial *pin;        // OUT_FINAL, optional
    void *out;
    spd_dtype out_dtype;
    int32_t epoch;                 // id of the call (both halves of a chained step share one)
    int32_t *status_words;         // where the kernel raises its status; null = the workspace header
    const spd_watch *watch;        // optional monitor of a private token range
    int plan_mode;                 // PlanMode: derive per call (default), derive and store, or load the stored plan
    bool plain_order;              // launch in plain stream order (an input was written by the kernel just before)
    const void *k_new, *v_new;     // optional append of the new token's rows to part[1] inside the launch
    bool wait_first;               // read nothing before the previous kernel on the stream has finished, not even a stored plan
    const spd_shape *layout_shape; // shape that lays the workspace out, if not `shape` (a call served in two halves keeps the whole batch's layout)
};

// The stored plan of a call is tagged with what it was cut for besides the lengths, so that a launch told to load a
// plan which was never stored (or stored for another shape) reports SPD_ERR_PLAN instead of using it.
int32_t plan_tag_of(const spd_shape &s, int min_tiles, int uniform) {
    uint32_t h = 0x9e3779b9u;
    const int32_t v[] = {s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim, static_cast<int32_t>(s.dtype), min_tiles, uniform};
    for (int32_t x : v) h = (h ^ static_cast<uint32_t>(x)) * 0x01000193u + 0x7f4a7c15u;
    h &= 0x7fffffffu;
    return static_cast<int32_t>(h ? h : 1u);
}

spd_status run_job(const Job &job, void *ws, size_t ws_bytes, void *stream) {
    const spd_shape &s = *job.shape;
    DeviceInfo di;
    spd_status rc = device_info(&di);
    if (rc != SPD_OK) return rc;
    const WsLayout L = ws_layout(job.layout_shape ? *job.layout_shape : s, di.sms);
    if (!ws || misaligned(ws, 256)) return SPD_ERR_INVALID_ARG;
    if (ws_bytes < L.total) return SPD_ERR_WORKSPACE;
    if (!job.q || misaligned(job.q, 16)) return SPD_ERR_INVALID_ARG;
    uint8_t *w = static_cast<uint8_t *>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    Params p;
    memset(&p, 0, sizeof p);
    p.B = s.batch; p.Hq = s.num_q_heads; p.Hkv = s.num_kv_heads; p.g = p.Hq / p.Hkv;
    p.hgroups = p.g > kHeadsPerItem ? p.g / kHeadsPerItem : 1;
    p.geff = p.g > kHeadsPerItem ? kHeadsPerItem : p.g;
    p.S = p.Hkv * p.hgroups;
    p.sm_scale = s.sm_scale;
    p.q = job.q;
    const bool bf = s.dtype == SPD_BF16;
    p.hdr = job.status_words ? job.status_words : reinterpret_cast<int32_t *>(w + L.hdr);
    p.bad = reinterpret_cast<int32_t *>(w + L.bad);
    p.tickets = reinterpret_cast<int32_t *>(w + L.tickets);
    p.rates = reinterpret_cast<float2 *>(w + L.rates);
    const int slot = (job.part[0] ? 1 : 0) + (job.part[1] ? 2 : 0) - 1;   // one stored plan per kind of call
    if (slot < 0) return SPD_ERR_INVALID_ARG;
    bool early_plan = false;
    p.rate_sel = static_cast<int32_t>(register_launch(ws, slot, job.plan_mode, &early_plan));   // rotates through the thirds
    p.plan_early = early_plan && !job.wait_first ? 1 : 0;
    p.min_tiles = g_min_tiles.load();
    p.uniform = g_uniform_shares.load();
    p.plan = reinterpret_cast<int32_t *>(w + L.plan + slot * kPlanBytes);
    p.plan_mode = job.plan_mode;
    p.plan_tag = plan_tag_of(s, p.min_tiles, p.uniform);
    p.epoch = job.epoch;
    p.scratch = reinterpret_cast<float *>(w + L.scratch);
    p.mode = job.mode;
    p.po = job.pout.o; p.pm = job.pout.m; p.pl = job.pout.l;
    if (job.pin) { p.in_o = job.pin->o; p.in_m = job.pin->m; p.in_l = job.pin->l; }
    p.out = job.out;
    p.out_bf16 = job.out_dtype == SPD_BF16;
    if (job.watch) { p.watch_lo = job.watch->tok_lo; p.watch_hi = job.watch->tok_hi; p.watch_out = job.watch->out; }
    if (job.k_new) {
        if (!job.part[1] || !job.v_new || job.part[1]->num_pages <= 0 || misaligned(job.k_new, 16) || misaligned(job.v_new, 16))
            return SPD_ERR_INVALID_ARG;
        p.k_new = static_cast<const uint8_t *>(job.k_new);
        p.v_new = static_cast<const uint8_t *>(job.v_new);
        // the append writes through pointers that spd_paged_kv declares const for the readers
        p.k_pool_w = static_cast<uint8_t *>(const_cast<void *>(job.part[1]->k_pool));
        p.v_pool_w = static_cast<uint8_t *>(const_cast<void *>(job.part[1]->v_pool));
        p.lens_w = const_cast<int32_t *>(job.part[1]->seq_lens);
    }

    CUtensorMap maps[4];
    int have = -1;
    for (int i = 0; i < 2; ++i) {
        const spd_paged_kv *kv = job.part[i];
        if (!kv) continue;
        p.part[i].indptr = kv->page_indptr;
        p.part[i].indices = kv->page_indices;
        p.part[i].lens = kv->seq_lens;
        p.part[i].num_pages = kv->num_pages;
        p.part[i].present = 1;
        if (kv->num_pages > 0) {
            if ((rc = make_map(&maps[2 * i], s, kv->k_pool, kv->num_pages)) != SPD_OK) return rc;
            if ((rc = make_map(&maps[2 * i + 1], s, kv->v_pool, kv->num_pages)) != SPD_OK) return rc;
            have = i;
        }
    }
    for (int i = 0; i < 2 && have >= 0; ++i)   // a partition without pages borrows a descriptor it never uses
        if (!job.part[i] || job.part[i]->num_pages == 0) {
            maps[2 * i] = maps[2 * have];
            maps[2 * i + 1] = maps[2 * have + 1];
        }

    if (have < 0) {
        // no partition owns a page: the kernel still runs (it writes the empty results), with
        // descriptors it never uses
        memset(maps, 0, sizeof maps);
    }
    int pj = -1;
    {
        std::lock_guard<std::mutex> lock(g_prof.mu);
        if (g_prof.on && g_prof.jobs < g_prof.cap) pj = g_prof.jobs++;
    }
    prof_mark(pj, 0, st);
    const int D = s.head_dim;
    const bool pdl = programmatic_launch() && !job.plain_order;
    if (bf && g_bf16_math.load() == 1) {
#define SPD_SIMT_CASE(DD, GG) if (D == DD && p.geff == GG) rc = launch_attn<MathBF16Simt<DD, GG>>(p, maps, di.sms, st, pdl);
        SPD_SIMT_CASE(64, 1) SPD_SIMT_CASE(64, 2) SPD_SIMT_CASE(64, 4) SPD_SIMT_CASE(64, 8)
        SPD_SIMT_CASE(128, 1) SPD_SIMT_CASE(128, 2) SPD_SIMT_CASE(128, 4) SPD_SIMT_CASE(128, 8)
#undef SPD_SIMT_CASE
    } else if (bf) {
        rc = D == 128 ? launch_attn<MathBF16<128>>(p, maps, di.sms, st, pdl) : launch_attn<MathBF16<64>>(p, maps, di.sms, st, pdl);
    } else {
#define SPD_F32_CASE(DD, GG) if (D == DD && p.geff == GG) rc = launch_attn<MathF32<DD, GG>>(p, maps, di.sms, st, pdl);
        SPD_F32_CASE(64, 1) SPD_F32_CASE(64, 2) SPD_F32_CASE(64, 4) SPD_F32_CASE(64, 8)
        SPD_F32_CASE(128, 1) SPD_F32_CASE(128, 2) SPD_F32_CASE(128, 4) SPD_F32_CASE(128, 8)
#undef SPD_F32_CASE
    }
    prof_mark(pj, 1, st);
    return rc;
}

spd_partial ws_partial(const spd_shape &s, void *ws, int sms) {
    const WsLayout L = ws_layout(s, sms);
    uint8_t *w = static_cast<uint8_t *>(ws);
    spd_partial part;
    part.o = reinterpret_cast<float *>(w + L.partial_o);
    part.m = reinterpret_cast<float *>(w + L.partial_m);
    part.l = reinterpret_cast<float *>(w + L.partial_l);
    return part;
}

}  // namespace

extern "C" {

spd_status spd_workspace_size(const spd_shape *shape, size_t *bytes) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (!bytes) return SPD_ERR_INVALID_ARG;
    DeviceInfo di;
    if ((rc = device_info(&di)) != SPD_OK) return rc;
    *bytes = ws_layout(*shape, di.sms).total;
    return SPD_OK;
}

static spd_status check_plan(int32_t plan) {
    return (plan == SPD_PLAN_PER_CALL || plan == SPD_PLAN_STORE || plan == SPD_PLAN_REUSE) ? SPD_OK : SPD_ERR_INVALID_ARG;
}

static spd_status partial_attn_impl(const spd_shape *shape, const void *q, const spd_paged_kv *priv, spd_partial out,
                                    int plan, void *ws, size_t ws_bytes, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if ((rc = check_kv(shape, priv)) != SPD_OK) return rc;
    if (!out.o || !out.m || !out.l || misaligned(out.o, 16)) return SPD_ERR_INVALID_ARG;
    Job job{};
    job.shape = shape; job.q = q; job.part[0] = priv; job.part[1] = nullptr;
    job.mode = OUT_PARTIAL; job.pout = out; job.pin = nullptr; job.out = nullptr; job.out_dtype = SPD_F32;
    job.epoch = next_epoch();
    job.plan_mode = plan;
    return run_job(job, ws, ws_bytes, cuda_stream);
}

static spd_status service_attn_merge_impl(const spd_shape *shape, const void *q, const spd_paged_kv *pub, spd_partial in,
                                          void *out, spd_dtype out_dtype, int plan, void *ws, size_t ws_bytes,
                                          void *cuda_stream, const void *k_new = nullptr, const void *v_new = nullptr) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if ((rc = check_kv(shape, pub)) != SPD_OK) return rc;
    if (!in.o || !in.m || !in.l || misaligned(in.o, 16)) return SPD_ERR_INVALID_ARG;
    if (!out || misaligned(out, 16)) return SPD_ERR_INVALID_ARG;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    Job job{};
    job.shape = shape; job.q = q; job.part[0] = nullptr; job.part[1] = pub;
    job.mode = OUT_FINAL; job.pin = &in; job.out = out; job.out_dtype = out_dtype;
    job.epoch = next_epoch();
    job.plan_mode = plan;
    if (k_new) {     // an appending launch reads lengths that the previous call of its kind bumps as its last act
        job.k_new = k_new; job.v_new = v_new;
        job.plain_order = true;
        job.wait_first = true;
    }
    return run_job(job, ws, ws_bytes, cuda_stream);
}

static spd_status decode_step_impl(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                   const spd_paged_kv *pub, void *out, spd_dtype out_dtype, int32_t fused, int plan,
                                   bool plain_order, void *ws, size_t ws_bytes, void *cuda_stream,
                                   const void *k_new = nullptr, const void *v_new = nullptr, bool wait_first = false) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if ((rc = check_kv(shape, priv)) != SPD_OK) return rc;
    if ((rc = check_kv(shape, pub)) != SPD_OK) return rc;
    if (!out || misaligned(out, 16)) return SPD_ERR_INVALID_ARG;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    if (fused) {
        Job job{};
        job.shape = shape; job.q = q; job.part[0] = priv; job.part[1] = pub;
        job.mode = OUT_FINAL; job.pin = nullptr; job.out = out; job.out_dtype = out_dtype;
        job.epoch = next_epoch();
        job.plan_mode = plan;
        job.plain_order = plain_order;
        job.k_new = k_new; job.v_new = v_new;
        job.wait_first = wait_first;
        return run_job(job, ws, ws_bytes, cuda_stream);
    }
    if (k_new) return SPD_ERR_UNSUPPORTED;      // the append rides on the fused step only
    DeviceInfo di;
    if ((rc = device_info(&di)) != SPD_OK) return rc;
    if (!ws || misaligned(ws, 256)) return SPD_ERR_INVALID_ARG;
    if (ws_bytes < ws_layout(*shape, di.sms).total) return SPD_ERR_WORKSPACE;
    // Both halves carry one call id, so a user flagged in the first half stays zeroed in the second.
    const spd_partial mid = ws_partial(*shape, ws, di.sms);
    Job a{}, b{};
    a.shape = b.shape = shape; a.q = b.q = q;
    a.part[0] = priv; a.mode = OUT_PARTIAL; a.pout = mid; a.out_dtype = SPD_F32;
    b.part[1] = pub; b.mode = OUT_FINAL; b.pin = &mid; b.out = out; b.out_dtype = out_dtype;
    a.epoch = b.epoch = next_epoch();
    a.plan_mode = b.plan_mode = plan;     // each half has a stored plan of its own
    a.plain_order = plain_order;
    if ((rc = run_job(a, ws, ws_bytes, cuda_stream)) != SPD_OK) return rc;
    return run_job(b, ws, ws_bytes, cuda_stream);
}

spd_status spd_partial_attn(const spd_shape *shape, const void *q, const spd_paged_kv *priv, spd_partial out,
                            void *ws, size_t ws_bytes, void *cuda_stream) {
    return partial_attn_impl(shape, q, priv, out, PLAN_DERIVE, ws, ws_bytes, cuda_stream);
}

spd_status spd_service_attn_merge(const spd_shape *shape, const void *q, const spd_paged_kv *pub, spd_partial in,
                                  void *out, spd_dtype out_dtype, void *ws, size_t ws_bytes, void *cuda_stream) {
    return service_attn_merge_impl(shape, q, pub, in, out, out_dtype, PLAN_DERIVE, ws, ws_bytes, cuda_stream);
}

spd_status spd_decode_step(const spd_shape *shape, const void *q, const spd_paged_kv *priv, const spd_paged_kv *pub,
                           void *out, spd_dtype out_dtype, int32_t fused, void *ws, size_t ws_bytes,
                           void *cuda_stream) {
    return decode_step_impl(shape, q, priv, pub, out, out_dtype, fused, PLAN_DERIVE, false, ws, ws_bytes, cuda_stream);
}

spd_status spd_partial_attn_planned(const spd_shape *shape, const void *q, const spd_paged_kv *priv, spd_partial out,
                                    spd_plan_mode plan, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (check_plan(plan) != SPD_OK) return SPD_ERR_INVALID_ARG;
    return partial_attn_impl(shape, q, priv, out, plan, ws, ws_bytes, cuda_stream);
}

spd_status spd_service_attn_merge_planned(const spd_shape *shape, const void *q, const spd_paged_kv *pub,
                                          spd_partial in, void *out, spd_dtype out_dtype, spd_plan_mode plan, void *ws,
                                          size_t ws_bytes, void *cuda_stream) {
    if (check_plan(plan) != SPD_OK) return SPD_ERR_INVALID_ARG;
    return service_attn_merge_impl(shape, q, pub, in, out, out_dtype, plan, ws, ws_bytes, cuda_stream);
}

spd_status spd_decode_step_append(const spd_shape *shape, const void *q, const void *k_new, const void *v_new,
                                  const spd_paged_kv *priv, const spd_paged_kv *pub, void *out, spd_dtype out_dtype,
                                  spd_plan_mode plan, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (check_plan(plan) != SPD_OK || !k_new || !v_new) return SPD_ERR_INVALID_ARG;
    // The kernel before this one on the stream may be the previous call of this very function on the same cache,
    // which adds one to the lengths as its last act: nothing is read before that kernel has finished.
    return decode_step_impl(shape, q, priv, pub, out, out_dtype, 1, plan, true, ws, ws_bytes, cuda_stream, k_new, v_new,
                            true);
}

spd_status spd_service_attn_merge_append(const spd_shape *shape, const void *q, const void *k_new, const void *v_new,
                                         const spd_paged_kv *pub, spd_partial in, void *out, spd_dtype out_dtype,
                                         spd_plan_mode plan, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (check_plan(plan) != SPD_OK || !k_new || !v_new) return SPD_ERR_INVALID_ARG;
    return service_attn_merge_impl(shape, q, pub, in, out, out_dtype, plan, ws, ws_bytes, cuda_stream, k_new, v_new);
}

spd_status spd_decode_step_planned(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                   const spd_paged_kv *pub, void *out, spd_dtype out_dtype, int32_t fused,
                                   spd_plan_mode plan, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (check_plan(plan) != SPD_OK) return SPD_ERR_INVALID_ARG;
    return decode_step_impl(shape, q, priv, pub, out, out_dtype, fused, plan, false, ws, ws_bytes, cuda_stream);
}

static spd_status check_watch(const spd_watch *w) {
    if (!w || !w->tok_lo || !w->tok_hi || !w->out) return SPD_ERR_INVALID_ARG;
    return SPD_OK;
}

spd_status spd_partial_attn_watch(const spd_shape *shape, const void *q, const spd_paged_kv *priv, spd_partial out,
                                  const spd_watch *watch, void *ws, size_t ws_bytes, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if ((rc = check_kv(shape, priv)) != SPD_OK) return rc;
    if ((rc = check_watch(watch)) != SPD_OK) return rc;
    if (!out.o || !out.m || !out.l || misaligned(out.o, 16)) return SPD_ERR_INVALID_ARG;
    Job job{};
    job.shape = shape; job.q = q; job.part[0] = priv;
    job.mode = OUT_PARTIAL; job.pout = out; job.out_dtype = SPD_F32;
    job.epoch = next_epoch();
    job.watch = watch;
    return run_job(job, ws, ws_bytes, cuda_stream);
}

spd_status spd_decode_step_watch(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                 const spd_paged_kv *pub, void *out, spd_dtype out_dtype, const spd_watch *watch,
                                 void *ws, size_t ws_bytes, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if ((rc = check_kv(shape, priv)) != SPD_OK) return rc;
    if ((rc = check_kv(shape, pub)) != SPD_OK) return rc;
    if ((rc = check_watch(watch)) != SPD_OK) return rc;
    if (!out || misaligned(out, 16)) return SPD_ERR_INVALID_ARG;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    Job job{};
    job.shape = shape; job.q = q; job.part[0] = priv; job.part[1] = pub;
    job.mode = OUT_FINAL; job.out = out; job.out_dtype = out_dtype;
    job.epoch = next_epoch();
    job.watch = watch;
    return run_job(job, ws, ws_bytes, cuda_stream);
}

spd_status spd_watch_alarm(const float *mass, int32_t batch, int32_t num_q_heads, const uint8_t *head_mask, float threshold,
                           int32_t *alarm, float *score) {
    if (!mass || !alarm || batch <= 0 || num_q_heads <= 0 || !(threshold == threshold)) return SPD_ERR_INVALID_ARG;
    for (int32_t u = 0; u < batch; ++u) {
        double sum = 0.0;
        int32_t n = 0;
        for (int32_t h = 0; h < num_q_heads; ++h)
            if (!head_mask || head_mask[h]) { sum += mass[static_cast<size_t>(u) * num_q_heads + h]; ++n; }
        const double mean = n ? sum / n : 0.0;
        if (score) score[u] = static_cast<float>(mean);
        alarm[u] = (n == 0 || !(mean >= static_cast<double>(threshold))) ? 1 : 0;     // NaN compares false: alarm
    }
    return SPD_OK;
}

// [T][H][128] bf16 as a 3-D tensor map; one box = `rows` tokens x 64 channels of one head, 128-byte swizzle.
static spd_status make_prompt_map(CUtensorMap *map, const void *ptr, int64_t T, int heads, int rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SPD_ERR_CUDA;
    cuuint64_t dims[3] = {128, static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(T)};
    cuuint64_t strides[2] = {128 * 2, static_cast<cuuint64_t>(heads) * 128 * 2};
    cuuint32_t box[3] = {64, 1, static_cast<cuuint32_t>(rows)};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SPD_OK : SPD_ERR_CUDA;
}

spd_status spd_prefill_attn(const spd_shape *shape, int64_t total_tokens, const void *q, const void *k, const void *v,
                            const int32_t *tok_indptr, void *k_pool, void *v_pool, int32_t num_pages,
                            const int32_t *page_indptr, const int32_t *page_indices, int32_t *seq_lens, void *out,
                            spd_dtype out_dtype, void *ws, size_t ws_bytes, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (!(shape->sm_scale > 0.f)) return SPD_ERR_UNSUPPORTED;   // the tensor-core kernels take row maxima before scaling
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    if (total_tokens < 0 || total_tokens >= (1ll << 31) - kPfBlock) return SPD_ERR_INVALID_ARG;
    if (!tok_indptr || !page_indptr || !seq_lens || !ws || misaligned(ws, 256)) return SPD_ERR_INVALID_ARG;
    if (ws_bytes < HDR_WORDS * 4) return SPD_ERR_WORKSPACE;
    if (total_tokens > 0 && (!q || !k || !v || !out || !k_pool || !v_pool || num_pages <= 0)) return SPD_ERR_INVALID_ARG;
    if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out, 16) || misaligned(k_pool, 128) ||
        misaligned(v_pool, 128))
        return SPD_ERR_INVALID_ARG;
    DeviceInfo di;
    if ((rc = device_info(&di)) != SPD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t T = total_tokens;

    PromptKvParams kp;
    kp.B = shape->batch; kp.Hkv = shape->num_kv_heads; kp.T = T;
    kp.row_bytes = shape->head_dim * (shape->dtype == SPD_BF16 ? 2 : 4);
    kp.k = static_cast<const uint8_t *>(k); kp.v = static_cast<const uint8_t *>(v); kp.tok_indptr = tok_indptr;
    kp.k_pool = static_cast<uint8_t *>(k_pool); kp.v_pool = static_cast<uint8_t *>(v_pool); kp.num_pages = num_pages;
    kp.page_indptr = page_indptr; kp.page_indices = page_indices; kp.lens = seq_lens; kp.hdr = static_cast<int32_t *>(ws);
    prompt_kv_kernel<<<static_cast<unsigned>(T + 1), 128, 0, st>>>(kp);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return SPD_ERR_CUDA;
    if (T == 0) return SPD_OK;

    PrefillParams pp;
    pp.B = shape->batch; pp.Hq = shape->num_q_heads; pp.Hkv = shape->num_kv_heads; pp.T = T;
    pp.sm_scale = shape->sm_scale; pp.tok_indptr = tok_indptr; pp.out = out; pp.out_bf16 = out_dtype == SPD_BF16;
    pp.hdr = static_cast<int32_t *>(ws);
    // fp32 prompts and head_dim 64 run on the FMA pipes (so does any shape when spd_set_prefill_rows(8) asks for it);
    // bf16 with head_dim 128, the shape that matters for throughput, runs on the tensor cores
    if (shape->dtype != SPD_BF16 || shape->head_dim != 128 || g_prefill_rows.load() == kFmaRows) {
        const int64_t max_blocks = (T + kFmaRows - 1) / kFmaRows + shape->batch;
        if (max_blocks >= (1ll << 31)) return SPD_ERR_UNSUPPORTED;
        dim3 grid(static_cast<unsigned>(max_blocks), static_cast<unsigned>(shape->num_q_heads));
        const bool bf = shape->dtype == SPD_BF16;
        const int D = shape->head_dim;
        if (bf && D == 128) prefill_fma_kernel<__nv_bfloat16, 128><<<grid, kFmaRows * 32, 0, st>>>(pp, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k), static_cast<const __nv_bfloat16 *>(v));
        else if (bf) prefill_fma_kernel<__nv_bfloat16, 64><<<grid, kFmaRows * 32, 0, st>>>(pp, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k), static_cast<const __nv_bfloat16 *>(v));
        else if (D == 128) prefill_fma_kernel<float, 128><<<grid, kFmaRows * 32, 0, st>>>(pp, static_cast<const float *>(q), static_cast<const float *>(k), static_cast<const float *>(v));
        else prefill_fma_kernel<float, 64><<<grid, kFmaRows * 32, 0, st>>>(pp, static_cast<const float *>(q), static_cast<const float *>(k), static_cast<const float *>(v));
        ++g_launches;
        return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ERR_CUDA;
    }

    // Long prompts go to the kernel with two 128-row tiles per CTA (each K/V block crosses from L2 once for
    // 256 rows); short ones to the one-tile kernel, whose CTAs are finer grained.  Only the mean length is
    // known on the host.
    const int rows_pref = g_prefill_rows.load();
    const bool pair = rows_pref == 256 || (rows_pref == 0 && T / shape->batch >= kPrefillPairFrom);
    CUtensorMap mq, mk, mv;
    if ((rc = make_prompt_map(&mq, q, T, shape->num_q_heads, kPfBlock)) != SPD_OK) return rc;
    if ((rc = make_prompt_map(&mk, k, T, shape->num_kv_heads, kPfKeys)) != SPD_OK) return rc;
    if ((rc = make_prompt_map(&mv, v, T, shape->num_kv_heads, kPfKeys)) != SPD_OK) return rc;
    static std::once_flag once[64];
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t attr_err = cudaSuccess;
    std::call_once(once[dev & 63], [&] {
        attr_err = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(prefill_smem_bytes()));
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(prefill_pair_smem_bytes()));
    });
    if (attr_err != cudaSuccess) return SPD_ERR_CUDA;
    const int rows = pair ? kPpRows : kPfBlock;
    const int64_t max_blocks = (T + rows - 1) / rows + shape->batch;   // >= sum over users of ceil(len / rows)
    dim3 grid(static_cast<unsigned>(max_blocks), static_cast<unsigned>(shape->num_q_heads));
    if (pair) prefill_pair_kernel<<<grid, kPpThreads, prefill_pair_smem_bytes(), st>>>(pp, mq, mk, mv);
    else prefill_kernel<<<grid, kPfThreads, prefill_smem_bytes(), st>>>(pp, mq, mk, mv);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ERR_CUDA;
}

spd_status spd_merge_partials(const spd_shape *shape, int32_t n, const spd_partial *parts, void *out,
                               spd_dtype out_dtype, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (n < 1 || n > kMaxMergeParts) return SPD_ERR_UNSUPPORTED;
    if (!parts || !out || misaligned(out, 16)) return SPD_ERR_INVALID_ARG;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    MergeParams mp;
    memset(&mp, 0, sizeof mp);
    mp.rows = shape->batch * shape->num_q_heads;
    mp.n = n;
    mp.out_bf16 = out_dtype == SPD_BF16;
    mp.out = out;
    for (int c = 0; c < n; ++c) {
        if (!parts[c].o || !parts[c].m || !parts[c].l || misaligned(parts[c].o, 16)) return SPD_ERR_INVALID_ARG;
        mp.o[c] = parts[c].o; mp.m[c] = parts[c].m; mp.l[c] = parts[c].l;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int blocks = (mp.rows + 3) / 4;
    if (shape->head_dim == 128) merge_partials_kernel<128><<<blocks, 128, 0, st>>>(mp);
    else merge_partials_kernel<64><<<blocks, 128, 0, st>>>(mp);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ERR_CUDA;
}

spd_status spd_append_kv(const spd_shape *shape, const void *k_new, const void *v_new, void *k_pool, void *v_pool,
                         int32_t num_pages, const int32_t *page_indptr, const int32_t *page_indices,
                         int32_t *seq_lens, void *ws, size_t ws_bytes, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (!k_new || !v_new || !k_pool || !v_pool || !page_indptr || !seq_lens || !ws || num_pages <= 0) return SPD_ERR_INVALID_ARG;
    if (misaligned(k_new, 16) || misaligned(v_new, 16) || misaligned(k_pool, 128) || misaligned(v_pool, 128) ||
        misaligned(ws, 256))
        return SPD_ERR_INVALID_ARG;
    if (ws_bytes < HDR_WORDS * 4) return SPD_ERR_WORKSPACE;
    AppendParams ap;
    ap.B = shape->batch; ap.Hkv = shape->num_kv_heads;
    ap.row_bytes = shape->head_dim * (shape->dtype == SPD_BF16 ? 2 : 4);
    ap.k_new = static_cast<const uint8_t *>(k_new); ap.v_new = static_cast<const uint8_t *>(v_new);
    ap.k_pool = static_cast<uint8_t *>(k_pool); ap.v_pool = static_cast<uint8_t *>(v_pool);
    ap.num_pages = num_pages; ap.indptr = page_indptr; ap.indices = page_indices; ap.lens = seq_lens;
    ap.hdr = static_cast<int32_t *>(ws);
    append_kernel<<<shape->batch, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(ap);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ERR_CUDA;
}

spd_status spd_token_step(const spd_shape *shape, int32_t num_layers, const spd_layer *layers, spd_dtype out_dtype,
                          int32_t same_lengths, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (!layers || num_layers <= 0) return SPD_ERR_INVALID_ARG;
    for (int32_t i = 0; i < num_layers; ++i) {
        const spd_layer &ly = layers[i];
        if (!ly.k_new || !ly.v_new) return SPD_ERR_INVALID_ARG;
        // With equal lengths in every layer the first layer's plan serves them all.  The first launch of the token
        // step starts in plain stream order (the kernel before it may be the previous token step's launch on the
        // same layer, which bumps the lengths this one reads); the others read their own layer's arrays, which
        // were last written a whole token step ago.
        const int plan = !same_lengths ? PLAN_DERIVE : (i == 0 ? PLAN_DERIVE_STORE : PLAN_LOAD);
        spd_status rc = decode_step_impl(shape, ly.q, &ly.priv, &ly.pub, ly.out, out_dtype, 1, plan, i == 0, ws, ws_bytes,
                                         cuda_stream, ly.k_new, ly.v_new);
        if (rc != SPD_OK) return rc;
    }
    return SPD_OK;
}

spd_status spd_step_blob_layout(const spd_shape *shape, int64_t priv_pages_listed, int64_t pub_pages_listed,
                                spd_dtype out_dtype, spd_step_blob *layout) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (!layout || priv_pages_listed < 0 || pub_pages_listed < 0) return SPD_ERR_INVALID_ARG;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    const size_t B = shape->batch, rows = B * shape->num_q_heads * shape->head_dim;
    const size_t es = shape->dtype == SPD_BF16 ? 2 : 4, oes = out_dtype == SPD_BF16 ? 2 : 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    layout->priv_pages_listed = priv_pages_listed;
    layout->pub_pages_listed = pub_pages_listed;
    layout->q = take(rows * es);
    layout->priv_indptr = take((B + 1) * 4);
    layout->priv_lens = take(B * 4);
    layout->priv_indices = take(static_cast<size_t>(priv_pages_listed) * 4);
    layout->pub_indptr = take((B + 1) * 4);
    layout->pub_lens = take(B * 4);
    layout->pub_indices = take(static_cast<size_t>(pub_pages_listed) * 4);
    layout->status = take(HDR_WORDS * 4);      // zero on the host: the upload clears the device copy
    layout->in_bytes = off;
    layout->out = take(rows * oes);
    layout->total_bytes = off;
    return SPD_OK;
}

spd_status spd_decode_step_host(const spd_shape *shape, const spd_step_blob *layout, void *host_blob,
                                void *device_blob, const spd_paged_kv *priv_pools, const spd_paged_kv *pub_pools,
                                spd_dtype out_dtype, int32_t *first_bad_user, void *ws, size_t ws_bytes,
                                void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    if (!layout || !host_blob || !device_blob || !priv_pools || !pub_pools || !ws) return SPD_ERR_INVALID_ARG;
    if (misaligned(device_blob, 256) || misaligned(host_blob, 16)) return SPD_ERR_INVALID_ARG;
    spd_step_blob want;
    if ((rc = spd_step_blob_layout(shape, layout->priv_pages_listed, layout->pub_pages_listed, out_dtype, &want)) != SPD_OK)
        return rc;
    if (memcmp(&want, layout, sizeof want) != 0) return SPD_ERR_INVALID_ARG;   // not a layout this library made
    const size_t B = shape->batch;
    const uint8_t *hb = static_cast<const uint8_t *>(host_blob);
    // the tables in the blob must fit the blob: their last prefix entry is the number of pages listed
    if (reinterpret_cast<const int32_t *>(hb + layout->priv_indptr)[B] > layout->priv_pages_listed ||
        reinterpret_cast<const int32_t *>(hb + layout->pub_indptr)[B] > layout->pub_pages_listed)
        return SPD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t *db = static_cast<uint8_t *>(device_blob);
    uint8_t *hbw = static_cast<uint8_t *>(host_blob);
    spd_paged_kv a = *priv_pools, b = *pub_pools;
    a.page_indptr = reinterpret_cast<const int32_t *>(db + layout->priv_indptr);
    a.seq_lens = reinterpret_cast<const int32_t *>(db + layout->priv_lens);
    a.page_indices = reinterpret_cast<const int32_t *>(db + layout->priv_indices);
    b.page_indptr = reinterpret_cast<const int32_t *>(db + layout->pub_indptr);
    b.seq_lens = reinterpret_cast<const int32_t *>(db + layout->pub_lens);
    b.page_indices = reinterpret_cast<const int32_t *>(db + layout->pub_indices);
    if ((rc = check_kv(shape, &a)) != SPD_OK || (rc = check_kv(shape, &b)) != SPD_OK) return rc;
    if (out_dtype != SPD_F32 && out_dtype != SPD_BF16) return SPD_ERR_UNSUPPORTED;
    const size_t row_in = static_cast<size_t>(shape->num_q_heads) * shape->head_dim * (shape->dtype == SPD_BF16 ? 2 : 4);
    const size_t row_out = static_cast<size_t>(shape->num_q_heads) * shape->head_dim * (out_dtype == SPD_BF16 ? 2 : 4);
    uint8_t *hs = hbw + layout->status;
    int32_t *hdr = reinterpret_cast<int32_t *>(hs);
    int32_t code = 0, bad_user = -1;

    // A large batch is served in parts so that the copies hide behind the kernels: while one part's kernel runs, the
    // next parts' q go up on a copy stream of the library's own and the previous part's output comes down.  The
    // tables of all parts travel with the first one.  Each part raises its status in words of its own of the blob's
    // status block.  Parts hold at least a megabyte of q or of output; smaller batches go as one.
    const size_t per_mb = ((row_in > row_out ? row_in : row_out) * B) >> 20;
    const int want_parts = per_mb >= 2 ? kHostStepParts : 1;
    const int parts = static_cast<size_t>(want_parts) <= B ? want_parts : 1;
    HostStepStreams hss;
    if (parts == 1 || host_step_streams(&hss) != SPD_OK) {
        if (cudaMemcpyAsync(db, hb, layout->in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SPD_ERR_CUDA;
        // The step raises its status in the blob (uploaded as zeros a moment ago), right in front of the
        // output, so that one copy brings both back.
        Job job{};
        job.shape = shape; job.q = db + layout->q; job.part[0] = &a; job.part[1] = &b;
        job.mode = OUT_FINAL; job.pin = nullptr; job.out = db + layout->out; job.out_dtype = out_dtype;
        job.epoch = next_epoch();
        job.status_words = reinterpret_cast<int32_t *>(db + layout->status);
        if ((rc = run_job(job, ws, ws_bytes, cuda_stream)) != SPD_OK) return rc;
        if (cudaMemcpyAsync(hs, db + layout->status, layout->total_bytes - layout->status, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return SPD_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return SPD_ERR_CUDA;
        code = hdr[HDR_STATUS];
        if (hdr[HDR_BAD_ENC]) bad_user = 0x7fffffff - hdr[HDR_BAD_ENC];
    } else {
        size_t first[kHostStepParts + 1];              // part i serves users [first[i], first[i + 1])
        for (int i = 0; i <= parts; ++i) first[i] = B * i / parts;
        const size_t q_all = B * row_in;
        // the first part's q, then everything behind q (tables of all parts, the zeroed status block), on the caller's stream
        if (cudaMemcpyAsync(db + layout->q, hb + layout->q, first[1] * row_in, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(db + layout->q + q_all, hb + layout->q + q_all, layout->in_bytes - (layout->q + q_all), cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SPD_ERR_CUDA;
        // the other parts' q on the copy stream, in order
        for (int i = 1; i < parts; ++i)
            if (cudaMemcpyAsync(db + layout->q + first[i] * row_in, hb + layout->q + first[i] * row_in, (first[i + 1] - first[i]) * row_in,
                                cudaMemcpyHostToDevice, hss.copy) != cudaSuccess ||
                cudaEventRecord(hss.q_up[i], hss.copy) != cudaSuccess)
                return SPD_ERR_CUDA;
        int32_t *status = reinterpret_cast<int32_t *>(db + layout->status);
        for (int i = 0; i < parts; ++i) {
            spd_shape si = *shape;
            si.batch = static_cast<int32_t>(first[i + 1] - first[i]);
            spd_paged_kv ai = a, bi = b;                // this part's users: the same tables, entered further in
            ai.page_indptr += first[i]; ai.seq_lens += first[i];
            bi.page_indptr += first[i]; bi.seq_lens += first[i];
            Job job{};
            job.shape = &si; job.q = db + layout->q + first[i] * row_in; job.part[0] = &ai; job.part[1] = &bi;
            job.mode = OUT_FINAL; job.out = db + layout->out + first[i] * row_out; job.out_dtype = out_dtype;
            job.epoch = next_epoch();
            job.status_words = status + 8 * i;
            job.layout_shape = shape;                   // every part lays the workspace out as the whole batch does
            if (i > 0 && cudaStreamWaitEvent(st, hss.q_up[i], 0) != cudaSuccess) return SPD_ERR_CUDA;
            if ((rc = run_job(job, ws, ws_bytes, cuda_stream)) != SPD_OK) return rc;
            if (i + 1 < parts) {                        // this part's output comes down under the next part's kernel
                if (cudaEventRecord(hss.done[i], st) != cudaSuccess || cudaStreamWaitEvent(hss.copy, hss.done[i], 0) != cudaSuccess ||
                    cudaMemcpyAsync(hbw + layout->out + first[i] * row_out, db + layout->out + first[i] * row_out,
                                    (first[i + 1] - first[i]) * row_out, cudaMemcpyDeviceToHost, hss.copy) != cudaSuccess)
                    return SPD_ERR_CUDA;
            }
        }
        const size_t last = first[parts - 1];
        if (cudaMemcpyAsync(hs, db + layout->status, HDR_WORDS * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaMemcpyAsync(hbw + layout->out + last * row_out, db + layout->out + last * row_out, (B - last) * row_out, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return SPD_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess || cudaStreamSynchronize(hss.copy) != cudaSuccess) return SPD_ERR_CUDA;
        for (int i = parts - 1; i >= 0; --i) {         // the lowest part that reports anything names the lowest user
            const int32_t c = hdr[8 * i + HDR_STATUS], enc = hdr[8 * i + HDR_BAD_ENC];
            if (c == SPD_ERR_TIMEOUT || (c != 0 && code != SPD_ERR_TIMEOUT)) code = c;
            if (enc) bad_user = static_cast<int32_t>(first[i]) + (0x7fffffff - enc);
        }
    }
    memset(hs, 0, HDR_WORDS * 4);              // ready for the next upload
    if (first_bad_user) *first_bad_user = bad_user;
    if (code == SPD_ERR_TIMEOUT) {             // a kernel that gave up may have left merge tickets drawn
        DeviceInfo di;
        if (device_info(&di) != SPD_OK) return SPD_ERR_CUDA;
        const WsLayout L = ws_layout(*shape, di.sms);
        if (cudaMemsetAsync(static_cast<uint8_t *>(ws) + L.tickets, 0, L.scratch - L.tickets, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return SPD_ERR_CUDA;
    }
    return static_cast<spd_status>(code);
}

spd_status spd_query_device_status(void *ws, void *cuda_stream, int32_t *first_bad_user) {
    if (!ws) return SPD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t hdr[8];
    if (cudaMemcpyAsync(hdr, ws, sizeof hdr, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPD_ERR_CUDA;
    if (first_bad_user) *first_bad_user = hdr[HDR_BAD_ENC] ? 0x7fffffff - hdr[HDR_BAD_ENC] : -1;
    if (hdr[HDR_STATUS] == 0) return SPD_OK;
    // clear the sticky words, the per-user flags and the tickets (a kernel that gave up on a wait may
    // have left tickets drawn)
    const WsHead H = ws_head(hdr[HDR_BATCH] > 0 ? hdr[HDR_BATCH] : 0, hdr[HDR_NSEQ] > 0 ? hdr[HDR_NSEQ] : 0);
    if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return SPD_ERR_CUDA;
    if (H.end > H.bad && cudaMemsetAsync(static_cast<uint8_t *>(ws) + H.bad, 0, H.end - H.bad, st) != cudaSuccess)
        return SPD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPD_ERR_CUDA;
    return static_cast<spd_status>(hdr[HDR_STATUS]);
}

int64_t spd_kernel_launch_count(void) { return g_launches.load(); }

spd_status spd_set_bf16_math(int32_t path) {
    if (path != 0 && path != 1) return SPD_ERR_INVALID_ARG;
    g_bf16_math.store(path);
    return SPD_OK;
}

spd_status spd_set_prefill_rows(int32_t rows) {
    if (rows != 0 && rows != 128 && rows != 256 && rows != kFmaRows) return SPD_ERR_INVALID_ARG;
    g_prefill_rows.store(rows);
    return SPD_OK;
}

spd_status spd_set_split(int32_t min_tiles_per_share, int32_t uniform_shares) {
    if (min_tiles_per_share < 0 || min_tiles_per_share > (1 << 30)) return SPD_ERR_INVALID_ARG;
    if (uniform_shares != 0 && uniform_shares != 1) return SPD_ERR_INVALID_ARG;
    g_min_tiles.store(min_tiles_per_share == 0 ? kMinTilesPerWarp : min_tiles_per_share);
    g_uniform_shares.store(uniform_shares);
    return SPD_OK;
}

spd_status spd_set_programmatic_launch(int32_t on) {
    if (on != 0 && on != 1) return SPD_ERR_INVALID_ARG;
    g_pdl.store(on);
    return SPD_OK;
}

spd_status spd_debug_read_plan(void *ws, int32_t which, void *cuda_stream, int32_t *tiles, int32_t *shares,
                               int32_t *bnd, int32_t bnd_capacity) {
    if (!ws || which < 0 || which >= kPlanSlots || bnd_capacity < 0 || (bnd_capacity > 0 && !bnd)) return SPD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const uint8_t *pl = static_cast<const uint8_t *>(ws) + ws_head(0, 0).plan + which * kPlanBytes;
    int32_t head[PLAN_HDR_WORDS];
    if (cudaMemcpyAsync(head, pl, sizeof head, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPD_ERR_CUDA;
    const int32_t A = head[PLAN_A];
    if (A < 0 || A > kMaxGrid * kMaxWarpsPerCta) return SPD_ERR_PLAN;
    if (tiles) *tiles = head[PLAN_T];
    if (shares) *shares = A;
    const int32_t nb = bnd_capacity < A + 1 ? bnd_capacity : A + 1;
    if (nb > 0) {
        if (cudaMemcpyAsync(bnd, pl + PLAN_BND * 4, static_cast<size_t>(nb) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return SPD_ERR_CUDA;
    }
    return SPD_OK;
}

spd_status spd_debug_sm_moves(void *ws, void *cuda_stream, int64_t *launches, int64_t *moves) {
    if (!ws) return SPD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t hdr[8];
    if (cudaMemcpyAsync(hdr, ws, sizeof hdr, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPD_ERR_CUDA;
    if (launches) *launches = hdr[HDR_SM_LAUNCHES];
    if (moves) *moves = hdr[HDR_SM_MOVES];
    return SPD_OK;
}

spd_status spd_profile_begin(int32_t max_calls) {
    if (max_calls <= 0 || max_calls > (1 << 16)) return SPD_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_prof.mu);
    while (static_cast<int>(g_prof.ev.size()) < 2 * max_calls) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return SPD_ERR_CUDA;
        g_prof.ev.push_back(e);
    }
    g_prof.cap = max_calls;
    g_prof.jobs = 0;
    g_prof.on = true;
    return SPD_OK;
}

spd_status spd_profile_end(int32_t *calls, double *kernel_ms) {
    std::lock_guard<std::mutex> lock(g_prof.mu);
    if (!g_prof.on) return SPD_ERR_INVALID_ARG;
    g_prof.on = false;
    double t = 0;
    for (int j = 0; j < g_prof.jobs; ++j) {
        float ms = 0.f;
        if (cudaEventSynchronize(g_prof.ev[2 * j + 1]) != cudaSuccess) return SPD_ERR_CUDA;
        if (cudaEventElapsedTime(&ms, g_prof.ev[2 * j], g_prof.ev[2 * j + 1]) != cudaSuccess) return SPD_ERR_CUDA;
        t += ms;
    }
    if (calls) *calls = g_prof.jobs;
    if (kernel_ms) *kernel_ms = t;
    return SPD_OK;
}

const char *spd_status_string(spd_status status) {
    switch (status) {
        case SPD_OK: return "ok";
        case SPD_ERR_INVALID_ARG: return "invalid argument";
        case SPD_ERR_UNSUPPORTED: return "unsupported shape, dtype or device";
        case SPD_ERR_WORKSPACE: return "workspace or staging buffer too small";
        case SPD_ERR_BAD_PAGE: return "page index or sequence length out of range (seen on the device)";
        case SPD_ERR_CUDA: return "CUDA call failed";
        case SPD_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case SPD_ERR_PLAN: return "no stored plan fits this call (never stored, or stored for another shape or grid)";
    }
    return "unknown status";
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Allocation-free variant: the workspace is a device array that lives in this library.
namespace {

// The name below is a host-side handle in host code, not a device address: only
// cudaGetSymbolAddress() turns it into a pointer that kernels and cudaMemset may use.
static __device__ __align__(256) unsigned char g_static_ws[SPD_STATIC_WS_BYTES];

// Device address of g_static_ws on the current device, looked up once per device.
spd_status static_ws_address(void **out) {
    static std::mutex mu;
    static void *addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) return SPD_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return SPD_OK;
}

}  // namespace

extern "C" spd_status spd_decode_step_static(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                             const spd_paged_kv *pub, void *out, spd_dtype out_dtype,
                                             int32_t wait_and_check, int32_t *first_bad_user, void *cuda_stream) {
    spd_status rc = check_shape(shape);
    if (rc != SPD_OK) return rc;
    DeviceInfo di;
    if ((rc = device_info(&di)) != SPD_OK) return rc;
    const WsLayout L = ws_layout(*shape, di.sms);
    if (L.total > SPD_STATIC_WS_BYTES) {
        fprintf(stderr, "spd_decode_step_static: this shape needs %zu bytes of workspace, the built-in array holds %u; "
                        "use spd_decode_step with a caller-provided workspace\n", L.total, SPD_STATIC_WS_BYTES);
        return SPD_ERR_WORKSPACE;
    }
    void *ws = nullptr;
    if ((rc = static_ws_address(&ws)) != SPD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array still holds the previous call's contents, laid out for the previous call's shape.  Three things
    // must start at zero: the sticky status words, the per-user flags and the merge tickets (this shape's ticket
    // region may lie where an earlier, smaller shape kept scratch floats, and a call that gave up on a wait leaves
    // tickets drawn).  The rest -- rate table, stored plans, scratch, the chained step's partial -- is either
    // rewritten before it is read or harmless when stale.
    if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return SPD_ERR_CUDA;
    if (cudaMemsetAsync(static_cast<uint8_t *>(ws) + L.bad, 0, L.scratch - L.bad, st) != cudaSuccess) return SPD_ERR_CUDA;
    rc = spd_decode_step(shape, q, priv, pub, out, out_dtype, 1, ws, SPD_STATIC_WS_BYTES, cuda_stream);
    if (rc != SPD_OK || !wait_and_check) return rc;
    return spd_query_device_status(ws, cuda_stream, first_bad_user);
}
