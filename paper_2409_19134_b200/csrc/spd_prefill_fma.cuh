// Prefill on the FMA pipes (protocol step 2; Fig. 3 step 0) for the shapes the tensor-core kernels do not take:
// fp32 prompts (head_dim 64 or 128, no reduced precision anywhere) and bf16 prompts with head_dim 64.  Causal
// self-attention over every user's prompt, softmax of sm_scale * q.k as in the decode kernels.
//
// One CTA = kFmaRows consecutive query rows of one (user, query head), one warp per row.  The rows share their keys:
// K and V come in blocks of 32 keys, widened to fp32, through shared memory (each element loaded once per CTA).  Per
// block every lane scores one key against its warp's query row, the warp takes maximum and sum with shuffles, and
// each lane accumulates head_dim / 32 channels of O.  Blocks of query rows are numbered as in the tensor-core kernels
// (prefill_find_block), so inconsistent token offsets are contained in the same way.
#pragma once

#include "spd_prefill.cuh"

namespace spd {

constexpr int kFmaRows = 8;     // query rows (warps) per CTA
constexpr int kFmaKeys = 32;    // keys per block: one per lane

template <typename T> __device__ __forceinline__ float fma_widen(T x);
template <> __device__ __forceinline__ float fma_widen<float>(float x) { return x; }
template <> __device__ __forceinline__ float fma_widen<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kFmaRows * 32) prefill_fma_kernel(PrefillParams p, const T *q, const T *k, const T *v) {
    constexpr int V = D / 32, KP = D + 1;          // K rows padded by one float: lane = key reads without bank conflicts
    __shared__ float Ks[kFmaKeys * KP];
    __shared__ float Vs[kFmaKeys * D];
    __shared__ float Qs[kFmaRows * D];
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / (p.Hq / p.Hkv);
    int qb, first, len;
    prefill_find_block(p, kFmaRows, blockIdx.x, lane, qb, first, len);
    if (qb < 0) return;                             // uniform over the CTA
    const int row = qb * kFmaRows + wid;            // this warp's query row within the prompt
    const bool live = row < len;
    if (live)
        for (int d = lane; d < D; d += 32) Qs[wid * D + d] = fma_widen<T>(q[(static_cast<int64_t>(first + row) * p.Hq + h) * D + d]);
    const int last_row = min(len, (qb + 1) * kFmaRows) - 1;     // keys 0 .. last_row are needed by somebody in the CTA
    const int nblocks = last_row / kFmaKeys + 1;
    float m = -INFINITY, l = 0.f, o[V];
#pragma unroll
    for (int i = 0; i < V; ++i) o[i] = 0.f;
    for (int jb = 0; jb < nblocks; ++jb) {
        __syncthreads();                            // the previous block's readers are done (and Qs is written)
        for (int idx = tid; idx < kFmaKeys * D; idx += kFmaRows * 32) {
            const int key = idx / D, d = idx - key * D, t = jb * kFmaKeys + key;
            float kk = 0.f, vv = 0.f;
            if (t <= last_row) {
                const int64_t src = (static_cast<int64_t>(first + t) * p.Hkv + kvh) * D + d;
                kk = fma_widen<T>(k[src]);
                vv = fma_widen<T>(v[src]);
            }
            Ks[key * KP + d] = kk;
            Vs[key * D + d] = vv;
        }
        __syncthreads();
        if (!live) continue;
        const int t = jb * kFmaKeys + lane;         // this lane's key
        float s = 0.f;
#pragma unroll 8
        for (int d = 0; d < D; ++d) s = fmaf(Qs[wid * D + d], Ks[lane * KP + d], s);
        s = t <= row ? s * p.sm_scale : -INFINITY;  // causal: token i attends to tokens 0..i
        float bm = s;
#pragma unroll
        for (int dd = 16; dd >= 1; dd >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, dd));
        if (bm == -INFINITY) continue;              // the whole block lies beyond this row's diagonal (warp-uniform)
        const float m_new = fmaxf(m, bm);
        const float alpha = expf(m - m_new);        // exp(-inf) = 0 on the first block
        const float pr = expf(s - m_new);
        float ps = pr;
#pragma unroll
        for (int dd = 16; dd >= 1; dd >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, dd);
        l = l * alpha + ps;
        m = m_new;
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] *= alpha;
        for (int j = 0; j < kFmaKeys; ++j) {
            const float pj = __shfl_sync(0xffffffffu, pr, j);
#pragma unroll
            for (int i = 0; i < V; ++i) o[i] = fmaf(pj, Vs[j * D + lane + 32 * i], o[i]);
        }
    }
    if (!live) return;
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int64_t dst = (static_cast<int64_t>(first + row) * p.Hq + h) * D;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const float y = o[i] * inv;
        if (p.out_bf16) reinterpret_cast<__nv_bfloat16 *>(p.out)[dst + lane + 32 * i] = __float2bfloat16_rn(y);
        else reinterpret_cast<float *>(p.out)[dst + lane + 32 * i] = y;
    }
}

}  // namespace spd
