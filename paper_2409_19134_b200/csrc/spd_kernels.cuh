// The kernel of the partitioned decode-attention path.
//
// One persistent launch does a whole call:
//   plan    : every CTA derives the same plan from memory nobody writes during the call --
//             validated page-tile counts per user, their prefix sums, and the share of the
//             flattened tile stream that each warp of the grid owns (sized by the streaming rate
//             each CTA showed on the previous call).
//   stream  : each warp streams its share of (user, kv head) page tiles from HBM through a
//             warp-private TMA ring in shared memory and keeps a running (O, m, l) per query head
//             (Sec. 4.2: m = max score, l = sum exp(s - m)).
//   merge   : a share that ends inside a sequence leaves its (O, m, l) in scratch and takes a
//             ticket; whoever delivers the last piece of a sequence recombines all of them
//             (Theorem 1 applied n-ways: M = max m_c, l = sum l_c e^{m_c-M}, O = sum O_c e^{m_c-M}).
//             Nobody waits for anybody.
//
// A "sequence" is the KV of one (user, kv head, group of <= 8 query heads): the private pages
// followed by the public pages (either part may be absent in a given call).
#pragma once

#include "spd_device.cuh"

namespace spd {

constexpr float kLog2e = 1.4426950408889634f;

// Shape of the bf16 attention CTA: warps per CTA and TMA ring depth per warp (8 KB per stage at
// head_dim 128).  warps * stages * 8 KB must fit the 227 KB of shared memory; at most 16 warps.
#ifndef SPD_BF16_WARPS
#define SPD_BF16_WARPS 8
#endif
#ifndef SPD_BF16_STAGES
#define SPD_BF16_STAGES 3
#endif

// ------------------------------------------------------------------------------------------------
// Validated page-tile counts of one user (private, public).  A pure function of the call's inputs,
// so every CTA that evaluates it agrees.  A user whose tables are inconsistent owns no tile and
// gets zeros; with Flag the user is also flagged for this call (a write to the workspace, so only
// done once the previous kernel on the stream has finished with it).
template <bool Flag = false>
__device__ __forceinline__ bool user_tiles(const Params &p, int u, int &n0, int &n1) {
    n0 = n1 = 0;
    bool bad = false;
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const PartDev &pt = p.part[s];
        if (!pt.present) continue;
        const int64_t lo = pt.indptr[u], hi = pt.indptr[u + 1], end = pt.indptr[p.B];
        const int64_t raw = pt.lens[u];
        const int64_t len = raw + ((s == 1 && p.k_new != nullptr) ? 1 : 0);   // an appending launch counts the new token
        if (lo < 0 || hi < lo || hi > end || raw < 0 || len > (hi - lo) * kPage ||
            (len > 0 && pt.indices == nullptr)) {
            bad = true;
        } else {
            const int n = static_cast<int>((len + kPage - 1) / kPage);
            if (s == 0) n0 = n; else n1 = n;
        }
    }
    if (bad) {
        n0 = n1 = 0;
        if (Flag) {
            p.bad[u] = p.epoch;
            flag_error(p.hdr, 4 /* SPD_ERR_BAD_PAGE */, u);
        }
    }
    return bad;
}

// ------------------------------------------------------------------------------------------------
// Last step for one (user, query head): either hand out the partial, or merge with the partial
// that came in (Theorem 1, both sides brought to the common maximum) and normalise.
// Each lane holds V = D/32 consecutive channels of O; m and l are warp-uniform.
template <int D>
__device__ __forceinline__ void finalize_store(const Params &p, int u, int h, float (&o)[D / 32], float m, float l,
                                               int lane, bool bad, float lw = 0.f) {
    constexpr int V = D / 32;
    const int64_t idx = static_cast<int64_t>(u) * p.Hq + h;
    if (p.mode == OUT_PARTIAL) {
        if (bad) {
#pragma unroll
            for (int i = 0; i < V; ++i) o[i] = 0.f;
            m = -INFINITY;
            l = 0.f;
        }
        float *dst = p.po + idx * D + lane * V;
        if constexpr (V == 4) *reinterpret_cast<float4 *>(dst) = make_float4(o[0], o[1], o[2], o[3]);
        else *reinterpret_cast<float2 *>(dst) = make_float2(o[0], o[1]);
        if (lane == 0) {
            p.pm[idx] = m;
            p.pl[idx] = l;
            if (p.watch_out) p.watch_out[idx] = bad ? 0.f : lw;   // same gauge as l: relative to m
        }
        return;
    }
    float L = l;
    float wself = 1.f;   // weight of this side after the merge with an incoming partial
    if (p.in_o != nullptr) {
        const float mi = p.in_m[idx], li = p.in_l[idx];
        const float M = fmaxf(m, mi);
        const float w = (m == -INFINITY) ? 0.f : expf(m - M);
        const float wi = (mi == -INFINITY) ? 0.f : expf(mi - M);
        const float *src = p.in_o + idx * D + lane * V;
        float oi[V];
        if constexpr (V == 4) { float4 t = *reinterpret_cast<const float4 *>(src); oi[0] = t.x; oi[1] = t.y; oi[2] = t.z; oi[3] = t.w; }
        else { float2 t = *reinterpret_cast<const float2 *>(src); oi[0] = t.x; oi[1] = t.y; }
        L = w * l + wi * li;
        wself = w;
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = w * o[i] + wi * oi[i];
    }
    const float inv = (L > 0.f && !bad) ? 1.f / L : 0.f;
    if (p.watch_out && lane == 0) p.watch_out[idx] = wself * lw * inv;   // share of the full softmax mass
#pragma unroll
    for (int i = 0; i < V; ++i) o[i] = (inv == 0.f) ? 0.f : o[i] * inv;
    if (p.out_bf16) {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + idx * D + lane * V;
#pragma unroll
        for (int i = 0; i < V; i += 2)
            *reinterpret_cast<__nv_bfloat162 *>(dst + i) = __floats2bfloat162_rn(o[i], o[i + 1]);
    } else {
        float *dst = reinterpret_cast<float *>(p.out) + idx * D + lane * V;
        if constexpr (V == 4) *reinterpret_cast<float4 *>(dst) = make_float4(o[0], o[1], o[2], o[3]);
        else *reinterpret_cast<float2 *>(dst) = make_float2(o[0], o[1]);
    }
}

__host__ __device__ constexpr int slot_floats(int D) { return kHeadsPerItem * D + 24; }   // O[8][D], m[8], l[8], watched l[8]

__device__ __forceinline__ int first_head(const Params &p, int sq) {
    const int kvh = sq / p.hgroups, hg = sq - kvh * p.hgroups;
    return kvh * p.g + hg * kHeadsPerItem;
}

// Scratch slot that warp w used for its piece of the sequence starting at tile s0: the first slot
// if the sequence contains the warp's first tile (bnd[w]), else the second.
__device__ __forceinline__ const float *piece_slot(const Params &p, int D, int w, const int32_t *bnd, int s0) {
    const int which = (bnd[w] >= s0) ? 0 : 1;
    return p.scratch + static_cast<int64_t>(2 * w + which) * slot_floats(D);
}

// The warp whose share [bnd[w], bnd[w+1]) holds tile t (shares may be empty; A = warps with a share).
__device__ __forceinline__ int warp_of_tile(const int32_t *bnd, int A, int t) {
    int lo = 0, hi = A;          // invariant: bnd[lo] <= t < bnd[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (bnd[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// Recombine the pieces that warps w_first..w_last left for one sequence (Theorem 1 applied n-ways,
// every piece brought to the common maximum) and finalise it.  Run by the warp that delivered the
// last piece.  Pieces are read past L1 (other SMs wrote them).  Lane c of a block of 32 pieces looks after the
// (m, l) of piece c; the O rows are fetched 16 at a time.  Every load here is a round trip to L2 on the critical
// path of a small call, so the first 16 O rows, the (m, l) values and the user's flag are requested together,
// before anything waits for any of them.
template <int D, int GE>
__device__ __noinline__ void merge_pieces(const Params &p, int u, int sq, int w_first, int w_last, const int32_t *bnd,
                                          int s0, int lane, bool bad) {
    constexpr int V = D / 32, H = kHeadsPerItem, PB = 16 / GE;   // PB pieces per batch of loads
    const int32_t flag = __ldcg(p.bad + u);      // used at the very end: was the user flagged by anybody during this call?
    float M[GE], L[GE], LW[GE], o[GE][V];
#pragma unroll
    for (int hh = 0; hh < GE; ++hh) {
        M[hh] = -INFINITY;
        L[hh] = 0.f;
        LW[hh] = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i) o[hh][i] = 0.f;
    }
    float x[PB][GE][V];
    auto load_rows = [&](int b0, int nb, int c0) {     // O rows of pieces [c0, c0 + PB) of the block that starts at warp b0
#pragma unroll
        for (int k = 0; k < PB; ++k) {
            const int c = c0 + k;
            const bool live = c < nb && bnd[b0 + c + 1] > bnd[b0 + c];
            const float *src = piece_slot(p, D, live ? b0 + c : b0, bnd, s0) + lane * V;
#pragma unroll
            for (int hh = 0; hh < GE; ++hh) {
                if constexpr (V == 4) {
                    const float4 t = live ? __ldcg(reinterpret_cast<const float4 *>(src + hh * D)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    x[k][hh][0] = t.x; x[k][hh][1] = t.y; x[k][hh][2] = t.z; x[k][hh][3] = t.w;
                } else {
                    const float2 t = live ? __ldcg(reinterpret_cast<const float2 *>(src + hh * D)) : make_float2(0.f, 0.f);
                    x[k][hh][0] = t.x; x[k][hh][1] = t.y;
                }
            }
        }
    };
    for (int b0 = w_first; b0 <= w_last; b0 += 32) {
        const int nb = min(32, w_last - b0 + 1);
        load_rows(b0, nb, 0);
        const bool mine = lane < nb && bnd[b0 + lane + 1] > bnd[b0 + lane];   // warps with an empty share left nothing
        const float *ms = piece_slot(p, D, mine ? b0 + lane : b0, bnd, s0) + H * D;
        float wgt[GE];
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
            const float mc = mine ? __ldcg(ms + hh) : -INFINITY;
            const float lc = mine ? __ldcg(ms + H + hh) : 0.f;
            const float lwc = (mine && p.watch_out) ? __ldcg(ms + 2 * H + hh) : 0.f;
            float mb = mc;
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, d));
            const float Mn = fmaxf(M[hh], mb);
            const float resc = (M[hh] == -INFINITY) ? 0.f : expf(M[hh] - Mn);
            wgt[hh] = (mc == -INFINITY) ? 0.f : expf(mc - Mn);
            float ls = wgt[hh] * lc, lws = wgt[hh] * lwc;
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                ls += __shfl_xor_sync(0xffffffffu, ls, d);
                lws += __shfl_xor_sync(0xffffffffu, lws, d);
            }
            L[hh] = L[hh] * resc + ls;
            LW[hh] = LW[hh] * resc + lws;
            M[hh] = Mn;
#pragma unroll
            for (int i = 0; i < V; ++i) o[hh][i] *= resc;
        }
        for (int c0 = 0; c0 < nb; c0 += PB) {
            if (c0 > 0) load_rows(b0, nb, c0);
#pragma unroll
            for (int k = 0; k < PB; ++k) {
                const int c = (c0 + k) & 31;
#pragma unroll
                for (int hh = 0; hh < GE; ++hh) {
                    const float wc = __shfl_sync(0xffffffffu, wgt[hh], c);   // a piece that is not live has weight 0
#pragma unroll
                    for (int i = 0; i < V; ++i) o[hh][i] = fmaf(wc, x[k][hh][i], o[hh][i]);
                }
            }
        }
    }
    const int hbase = first_head(p, sq);
    bad = bad || flag == p.epoch;
#pragma unroll
    for (int hh = 0; hh < GE; ++hh) finalize_store<D>(p, u, hbase + hh, o[hh], M[hh], L[hh], lane, bad, LW[hh]);
}

// A finished segment sits in shared memory as So[8][D+4], Sm[8], Sl[8], Sw[8] (Sw = watched part of l,
// right behind Sl).  A segment that is a whole
// sequence is finalised on the spot (the warp has seen every page of it, so `bad` is complete).
template <int D>
__device__ __forceinline__ void finalize_segment(const Params &p, const float *So, const float *Sm, const float *Sl,
                                                 int u, int sq, int lane, bool bad) {
    constexpr int V = D / 32, PITCH = D + 4;
    const int hbase = first_head(p, sq);
    for (int hh = 0; hh < p.geff; ++hh) {
        float o[V];
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = So[hh * PITCH + lane * V + i];
        finalize_store<D>(p, u, hbase + hh, o, Sm[hh], Sl[hh], lane, bad, Sl[kHeadsPerItem + hh]);
    }
}

// A segment that is only a piece of its sequence goes to scratch slot 2w (kind 1) or 2w+1 (kind 2).
// The stores are fire-and-forget; piece_ticket fences them before it draws the ticket.
template <int D>
__device__ __forceinline__ void piece_store(const Params &p, const float *So, const float *Sm, const float *Sl,
                                            int kind, int gwarp, int lane) {
    constexpr int V = D / 32, PITCH = D + 4;
    float *dst = p.scratch + static_cast<int64_t>(2 * gwarp + (kind - 1)) * slot_floats(D);
#pragma unroll
    for (int hh = 0; hh < kHeadsPerItem; ++hh) {
        if (hh >= p.geff) break;     // rows past the group are never read back
        if constexpr (V == 4)
            __stcg(reinterpret_cast<float4 *>(dst + hh * D + lane * V), *reinterpret_cast<const float4 *>(So + hh * PITCH + lane * V));
        else
            __stcg(reinterpret_cast<float2 *>(dst + hh * D + lane * V), *reinterpret_cast<const float2 *>(So + hh * PITCH + lane * V));
    }
    if (lane < 8) {
        __stcg(dst + kHeadsPerItem * D + lane, Sm[lane]);
        __stcg(dst + kHeadsPerItem * D + 8 + lane, Sl[lane]);
        __stcg(dst + kHeadsPerItem * D + 16 + lane, Sl[kHeadsPerItem + lane]);
    }
}

// A piece of a sequence: whose it is, the sequence's tile count and first tile, and whether a
// page of the piece was out of range.
struct PieceInfo {
    int u, sq, np, s0;
    bool bad;
};

// Draw the ticket of a piece already stored; the warp that draws the last ticket of a sequence
// merges all its pieces (and puts the counter back to zero for the next call).
template <int D>
__device__ __forceinline__ void piece_ticket(const Params &p, const PieceInfo &pp, const int32_t *bnd, int A, int lane) {
    const int w_first = warp_of_tile(bnd, A, pp.s0), w_last = warp_of_tile(bnd, A, pp.s0 + pp.np - 1);
    int pieces = 0;
    for (int w = w_first + lane; w <= w_last; w += 32) pieces += bnd[w + 1] > bnd[w] ? 1 : 0;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) pieces += __shfl_xor_sync(0xffffffffu, pieces, d);
    __threadfence();     // this lane's part of the piece is visible before the ticket is drawn
    __syncwarp();
    int ticket = 0;
    int32_t *counter = p.tickets + static_cast<int64_t>(pp.u) * p.S + pp.sq;
    if (lane == 0) ticket = atomicAdd(counter, 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket != pieces - 1) return;         // other pieces are still to come
    __threadfence();
    if (lane == 0) *counter = 0;              // everybody has drawn: ready for the next call
    switch (p.geff) {      // the user's flag (raised by anybody during this call) is looked up inside, with the pieces
        case 1: merge_pieces<D, 1>(p, pp.u, pp.sq, w_first, w_last, bnd, pp.s0, lane, pp.bad); break;
        case 2: merge_pieces<D, 2>(p, pp.u, pp.sq, w_first, w_last, bnd, pp.s0, lane, pp.bad); break;
        case 4: merge_pieces<D, 4>(p, pp.u, pp.sq, w_first, w_last, bnd, pp.s0, lane, pp.bad); break;
        default: merge_pieces<D, 8>(p, pp.u, pp.sq, w_first, w_last, bnd, pp.s0, lane, pp.bad); break;
    }
}

// ------------------------------------------------------------------------------------------------
// bf16 tile math on the tensor cores (mma.sync m16n8k16, fp32 accumulate).
//   S  = Q K^T   : M = 16 query-head rows (8 used), N = 8 tokens (x2), K = head_dim
//   O^T = V^T P^T : M = 16 channels (x D/16), N = 8 query heads, K = 16 tokens
// The accumulator fragment of S (row = head, columns = two consecutive tokens) is exactly the B
// fragment that the second product wants for P^T, so P never leaves registers.  P is split into a
// bf16 head and a bf16 remainder (two MMAs) so that rounding P to 8 bits of mantissa does not show
// in the output.  K and V tiles sit in shared memory as 128-byte-swizzled [half][16 tokens][64].
template <int D_>
struct MathBF16 {
    static constexpr int D = D_;
    static constexpr int kTileBytes = kPage * D * 2;
    static constexpr int kBoxes = D / 64;          // TMA boxes per tile (64 bf16 = 128 B wide)
    static constexpr int kBoxBytes = kPage * 128;
    static constexpr int kBoxCols = 64;
    static constexpr int kWarps = SPD_BF16_WARPS;
    static constexpr int kStages = SPD_BF16_STAGES;
    static constexpr int kExtraBytes = 0;
    static constexpr int KS = D / 16;
    // byte offset, inside a K or V tile in shared memory, of 16-byte chunk c of token row r
    __device__ static __forceinline__ int chunk_offset(int r, int c) { return (c >> 3) * kBoxBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4); }

    struct State {
        uint32_t qf[KS][2];
        float o[KS][4];
        float m, l;
        float lw;          // part of l that came from the watched token range
        int wlo, whi;      // watched range of the private partition, [wlo, whi); empty = not watching
    };

    __device__ static __forceinline__ void begin(State &st, const Params &p, int u, int sq, int lane, uint8_t *) {
        const int kvh = sq / p.hgroups, hg = sq - kvh * p.hgroups;
        const int row = lane >> 2;
        const bool live = row < p.geff;
        const int h = kvh * p.g + hg * kHeadsPerItem + row;
        const __nv_bfloat16 *qrow =
            reinterpret_cast<const __nv_bfloat16 *>(p.q) + (static_cast<int64_t>(u) * p.Hq + (live ? h : 0)) * D;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int d0 = ks * 16 + 2 * (lane & 3);
            st.qf[ks][0] = live ? *reinterpret_cast<const uint32_t *>(qrow + d0) : 0u;
            st.qf[ks][1] = live ? *reinterpret_cast<const uint32_t *>(qrow + d0 + 8) : 0u;
        }
#pragma unroll
        for (int mt = 0; mt < KS; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) st.o[mt][i] = 0.f;
        st.m = -INFINITY;
        st.l = 0.f;
        st.lw = 0.f;
        st.wlo = p.watch_out ? p.watch_lo[u] : 0;
        st.whi = p.watch_out ? p.watch_hi[u] : 0;
    }

    // watch_base: index within the private partition of the tile's first token (hugely negative for
    // a tile of the public partition, so that nothing of it counts as watched)
    __device__ static __forceinline__ void tile(State &st, const Params &p, uint8_t *Ks, uint8_t *Vs, int valid,
                                                int lane, uint8_t *, int watch_base) {
        const int mat = lane >> 3, r = lane & 7;
        const int tok = ((mat >> 1) << 3) + r;
        const uint32_t lane_off = tok * 128;
        const int csel = mat & 1;
        if (valid < kPage) {
            // V rows past the partition's end may hold anything (even NaN): zero them, since
            // 0 * NaN would poison the product.  Rows stay rows under the 128-byte swizzle.
            for (int i = lane; i < (kPage - valid) * 8 * kBoxes; i += 32) {
                const int rr = valid + (i >> 3) % (kPage - valid), rest = (i >> 3) / (kPage - valid);
                *reinterpret_cast<uint4 *>(Vs + rest * kBoxBytes + rr * 128 + (i & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
            __syncwarp();
        }
        const uint32_t kbase = smem_u32(Ks), vbase = smem_u32(Vs);
        float s[2][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) s[0][i] = s[1][i] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int c = 2 * (ks & 3) + csel;
            uint32_t b00, b01, b10, b11;
            ldsm_x4(kbase + (ks >> 2) * kBoxBytes + lane_off + ((c ^ r) << 4), b00, b10, b01, b11);
            // matrices: 0 = tokens 0-7 / chunk c, 1 = tokens 0-7 / chunk c+1, 2,3 = tokens 8-15
            mma_bf16(s[0], st.qf[ks][0], 0u, st.qf[ks][1], 0u, b00, b10);
            mma_bf16(s[1], st.qf[ks][0], 0u, st.qf[ks][1], 0u, b01, b11);
        }
        const int tk = 2 * (lane & 3);
        float v0 = s[0][0] * p.sm_scale, v1 = s[0][1] * p.sm_scale;
        float v2 = s[1][0] * p.sm_scale, v3 = s[1][1] * p.sm_scale;
        if (tk >= valid) v0 = -INFINITY;
        if (tk + 1 >= valid) v1 = -INFINITY;
        if (tk + 8 >= valid) v2 = -INFINITY;
        if (tk + 9 >= valid) v3 = -INFINITY;
        float tmax = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        const float m_new = fmaxf(st.m, tmax);
        const float alpha = ex2_approx((st.m - m_new) * kLog2e);
        const float p0 = ex2_approx((v0 - m_new) * kLog2e), p1 = ex2_approx((v1 - m_new) * kLog2e);
        const float p2 = ex2_approx((v2 - m_new) * kLog2e), p3 = ex2_approx((v3 - m_new) * kLog2e);
        st.l = st.l * alpha + ((p0 + p1) + (p2 + p3));
        st.m = m_new;
        if (st.whi > st.wlo) {   // warp-uniform
            const int t0 = watch_base + tk;
            float w = (t0 >= st.wlo && t0 < st.whi) ? p0 : 0.f;
            w += (t0 + 1 >= st.wlo && t0 + 1 < st.whi) ? p1 : 0.f;
            w += (t0 + 8 >= st.wlo && t0 + 8 < st.whi) ? p2 : 0.f;
            w += (t0 + 9 >= st.wlo && t0 + 9 < st.whi) ? p3 : 0.f;
            st.lw = st.lw * alpha + w;
        }
        const uint32_t bh0 = pack_bf16(p0, p1), bh1 = pack_bf16(p2, p3);
        const __nv_bfloat162 h0 = *reinterpret_cast<const __nv_bfloat162 *>(&bh0);
        const __nv_bfloat162 h1 = *reinterpret_cast<const __nv_bfloat162 *>(&bh1);
        const uint32_t bl0 = pack_bf16(p0 - __low2float(h0), p1 - __high2float(h0));
        const uint32_t bl1 = pack_bf16(p2 - __low2float(h1), p3 - __high2float(h1));
        // the accumulator columns are heads 2*(lane%4) and +1; their rescale factors live in the
        // quads that own those heads as rows
        const float ae = __shfl_sync(0xffffffffu, alpha, (lane & 3) * 8);
        const float ao = __shfl_sync(0xffffffffu, alpha, (lane & 3) * 8 + 4);
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            const int c = 2 * (mt & 3) + csel;
            uint32_t a0, a1, a2, a3;
            ldsm_x4_t(vbase + (mt >> 2) * kBoxBytes + lane_off + ((c ^ r) << 4), a0, a1, a2, a3);
            st.o[mt][0] *= ae; st.o[mt][2] *= ae;
            st.o[mt][1] *= ao; st.o[mt][3] *= ao;
            mma_bf16(st.o[mt], a0, a1, a2, a3, bh0, bh1);
            mma_bf16(st.o[mt], a0, a1, a2, a3, bl0, bl1);
        }
    }

    // Spill the running state into shared memory as So[8][D+4], Sm[8], Sl[8].
    __device__ static __forceinline__ void finish(State &st, float *So, float *Sm, float *Sl, int lane) {
        constexpr int PITCH = D + 4;
        const int hd = 2 * (lane & 3), dr = lane >> 2;
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            So[hd * PITCH + mt * 16 + dr] = st.o[mt][0];
            So[(hd + 1) * PITCH + mt * 16 + dr] = st.o[mt][1];
            So[hd * PITCH + mt * 16 + dr + 8] = st.o[mt][2];
            So[(hd + 1) * PITCH + mt * 16 + dr + 8] = st.o[mt][3];
        }
        float l = st.l, lw = st.lw;
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        lw += __shfl_xor_sync(0xffffffffu, lw, 1);
        lw += __shfl_xor_sync(0xffffffffu, lw, 2);
        if ((lane & 3) == 0) { Sm[lane >> 2] = st.m; Sl[lane >> 2] = l; Sl[kHeadsPerItem + (lane >> 2)] = lw; }
    }
};

// ------------------------------------------------------------------------------------------------
// bf16 tile math on the FMA pipes: the comparison arm for the tensor-core policy above (same tiles,
// same TMA descriptors, same 128-byte-swizzled layout in shared memory; only the arithmetic differs).
// K and V are widened to fp32 on the fly.  Costs grow with the group size, which is the point of the
// comparison: at one query head per KV head the FMA pipes keep up with HBM, at eight they do not.
template <int D_, int GE_>
struct MathBF16Simt {
    static constexpr int D = D_, GE = GE_;
    static constexpr int kTileBytes = kPage * D * 2;
    static constexpr int kBoxes = D / 64;
    static constexpr int kBoxBytes = kPage * 128;
    static constexpr int kBoxCols = 64;
    static constexpr int kWarps = 7;       // one fewer than the tensor-core policy: q and P need 4.6 KB per warp
    static constexpr int kStages = SPD_BF16_STAGES;
    static constexpr int kExtraBytes = (kHeadsPerItem * D + kHeadsPerItem * kPage) * 4;  // q (fp32), P
    static constexpr int V = D / 32;
    __device__ static __forceinline__ int chunk_offset(int r, int c) { return (c >> 3) * kBoxBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4); }

    struct State {
        float o[GE][V];
        float m[GE], l[GE], lw[GE];
        int wlo, whi;
    };

    __device__ static __forceinline__ void begin(State &st, const Params &p, int u, int sq, int lane, uint8_t *extra) {
        float *qs = reinterpret_cast<float *>(extra);
        const int hbase = first_head(p, sq);
        const __nv_bfloat16 *qg = reinterpret_cast<const __nv_bfloat16 *>(p.q) + (static_cast<int64_t>(u) * p.Hq + hbase) * D;
        __syncwarp();
        for (int i = lane; i < GE * D; i += 32) qs[i] = __bfloat162float(qg[i]);
        __syncwarp();
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) st.o[hh][i] = 0.f;
            st.m[hh] = -INFINITY;
            st.l[hh] = 0.f;
            st.lw[hh] = 0.f;
        }
        st.wlo = p.watch_out ? p.watch_lo[u] : 0;
        st.whi = p.watch_out ? p.watch_hi[u] : 0;
    }

    __device__ static __forceinline__ void tile(State &st, const Params &p, uint8_t *Ks, uint8_t *Vs, int valid,
                                                int lane, uint8_t *extra, int watch_base) {
        const float *qs = reinterpret_cast<const float *>(extra);
        float *Ps = reinterpret_cast<float *>(extra) + kHeadsPerItem * D;
        // scores: lane = (token t, half of head_dim); a half is 64 columns = one swizzled box (D = 128)
        // or half a box (D = 64); 16-byte chunk c of row t sits at chunk c ^ (t & 7) of its 128-byte line
        const int t = lane & 15, hf = lane >> 4;
        constexpr int NCH = D / 16;                       // chunks of 8 channels per half row
        const int chunk0 = (D == 128) ? 0 : hf * NCH;     // first chunk of this half within its box
        const uint8_t *kline = Ks + ((D == 128) ? hf * kBoxBytes : 0) + t * 128;
        float s[GE];
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) s[hh] = 0.f;
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int c = chunk0 + j;
            const uint4 raw = *reinterpret_cast<const uint4 *>(kline + ((c ^ (t & 7)) << 4));
            const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
            float kf[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(k2[i]); kf[2 * i] = f.x; kf[2 * i + 1] = f.y; }
#pragma unroll
            for (int hh = 0; hh < GE; ++hh) {
                const float4 qa = *reinterpret_cast<const float4 *>(qs + hh * D + hf * (D / 2) + 8 * j);
                const float4 qb = *reinterpret_cast<const float4 *>(qs + hh * D + hf * (D / 2) + 8 * j + 4);
                s[hh] = fmaf(kf[0], qa.x, s[hh]); s[hh] = fmaf(kf[1], qa.y, s[hh]);
                s[hh] = fmaf(kf[2], qa.z, s[hh]); s[hh] = fmaf(kf[3], qa.w, s[hh]);
                s[hh] = fmaf(kf[4], qb.x, s[hh]); s[hh] = fmaf(kf[5], qb.y, s[hh]);
                s[hh] = fmaf(kf[6], qb.z, s[hh]); s[hh] = fmaf(kf[7], qb.w, s[hh]);
            }
        }
        __syncwarp();   // the previous tile's readers of Ps are done
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
            float v = s[hh] + __shfl_xor_sync(0xffffffffu, s[hh], 16);
            v = (t < valid) ? v * p.sm_scale : -INFINITY;
            float tmax = v;
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, d));
            const float m_new = fmaxf(st.m[hh], tmax);
            const float alpha = ex2_approx((st.m[hh] - m_new) * kLog2e);
            const float pr = ex2_approx((v - m_new) * kLog2e);
            st.l[hh] = st.l[hh] * alpha + (hf == 0 ? pr : 0.f);
            st.lw[hh] = st.lw[hh] * alpha + ((hf == 0 && watch_base + t >= st.wlo && watch_base + t < st.whi) ? pr : 0.f);
            st.m[hh] = m_new;
#pragma unroll
            for (int i = 0; i < V; ++i) st.o[hh][i] *= alpha;
            if (hf == 0) Ps[hh * kPage + t] = pr;
        }
        __syncwarp();
        // P V: lane owns channels [lane * V, lane * V + V): V bf16 inside one 16-byte chunk
        const int col = lane * V;                                   // channel
        const int box = col / 64, cc = (col % 64) / 8, within = (col % 8) * 2;   // box, chunk, byte in chunk
        for (int tt = 0; tt < valid; ++tt) {   // rows past `valid` are never touched
            const uint8_t *src = Vs + box * kBoxBytes + tt * 128 + ((cc ^ (tt & 7)) << 4) + within;
            float vv[V];
            if constexpr (V == 4) {
                const uint2 raw = *reinterpret_cast<const uint2 *>(src);
                const __nv_bfloat162 *v2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
                const float2 a = __bfloat1622float2(v2[0]), b = __bfloat1622float2(v2[1]);
                vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
            } else {
                const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(src));
                vv[0] = a.x; vv[1] = a.y;
            }
#pragma unroll
            for (int hh = 0; hh < GE; ++hh) {
                const float pr = Ps[hh * kPage + tt];
#pragma unroll
                for (int i = 0; i < V; ++i) st.o[hh][i] = fmaf(pr, vv[i], st.o[hh][i]);
            }
        }
    }

    __device__ static __forceinline__ void finish(State &st, float *So, float *Sm, float *Sl, int lane) {
        constexpr int PITCH = D + 4;
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) So[hh * PITCH + lane * V + i] = st.o[hh][i];
            float l = st.l[hh], lw = st.lw[hh];
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) {
                l += __shfl_xor_sync(0xffffffffu, l, d);
                lw += __shfl_xor_sync(0xffffffffu, lw, d);
            }
            if (lane == 0) { Sm[hh] = st.m[hh]; Sl[hh] = l; Sl[kHeadsPerItem + hh] = lw; }
        }
        for (int hh = GE; hh < kHeadsPerItem; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) So[hh * PITCH + lane * V + i] = 0.f;
            if (lane == 0) { Sm[hh] = -INFINITY; Sl[hh] = 0.f; Sl[kHeadsPerItem + hh] = 0.f; }
        }
    }
};

// ------------------------------------------------------------------------------------------------
// fp32 tile math on the FMA pipes (no reduced precision anywhere).
//   scores : lane = (token t = lane & 15, half of head_dim = lane >> 4); each lane walks its half
//            row of K in float4 steps, starting at a chunk rotated by t so that the 8 lanes of a
//            shared-memory phase hit 8 different bank groups; halves are added with one shuffle.
//   P V    : probabilities go through a small shared array; each lane owns D/32 channels of O.
template <int D_, int GE_>
struct MathF32 {
    static constexpr int D = D_, GE = GE_;
    static constexpr int kTileBytes = kPage * D * 4;
    static constexpr int kBoxes = 1;
    static constexpr int kBoxBytes = kTileBytes;
    static constexpr int kBoxCols = D;
    static constexpr int kWarps = 4;
    static constexpr int kStages = D == 128 ? 2 : 3;   // 16 KB per stage at head_dim 128
    static constexpr int kExtraBytes = (kHeadsPerItem * D + kHeadsPerItem * kPage) * 4;  // q, P
    static constexpr int V = D / 32;
    __device__ static __forceinline__ int chunk_offset(int r, int c) { return r * D * 4 + c * 16; }

    struct State {
        float o[GE][V];
        float m[GE], l[GE], lw[GE];
        int wlo, whi;
    };

    __device__ static __forceinline__ void begin(State &st, const Params &p, int u, int sq, int lane, uint8_t *extra) {
        float *qs = reinterpret_cast<float *>(extra);
        const int kvh = sq / p.hgroups, hg = sq - kvh * p.hgroups;
        const int hbase = kvh * p.g + hg * kHeadsPerItem;
        const float *qg = reinterpret_cast<const float *>(p.q) + (static_cast<int64_t>(u) * p.Hq + hbase) * D;
        __syncwarp();
        for (int i = lane; i < GE * D; i += 32) qs[i] = qg[i];
        __syncwarp();
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) st.o[hh][i] = 0.f;
            st.m[hh] = -INFINITY;
            st.l[hh] = 0.f;
            st.lw[hh] = 0.f;
        }
        st.wlo = p.watch_out ? p.watch_lo[u] : 0;
        st.whi = p.watch_out ? p.watch_hi[u] : 0;
    }

    __device__ static __forceinline__ void tile(State &st, const Params &p, uint8_t *Ks, uint8_t *Vs, int valid,
                                                int lane, uint8_t *extra, int watch_base) {
        const float *qs = reinterpret_cast<const float *>(extra);
        float *Ps = reinterpret_cast<float *>(extra) + kHeadsPerItem * D;
        const int t = lane & 15, hf = lane >> 4;
        constexpr int HALF = D / 2, NCH = HALF / 4;
        const float *krow = reinterpret_cast<const float *>(Ks) + t * D + hf * HALF;
        float s[GE];
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) s[hh] = 0.f;
#pragma unroll(NCH > 8 ? 4 : NCH)      // head_dim 128: fully unrolled, sixteen steps times eight heads overflow the register file
        for (int j = 0; j < NCH; ++j) {
            const int c = (j + t) & (NCH - 1);
            const float4 k4 = *reinterpret_cast<const float4 *>(krow + 4 * c);
#pragma unroll
            for (int hh = 0; hh < GE; ++hh) {
                const float4 q4 = *reinterpret_cast<const float4 *>(qs + hh * D + hf * HALF + 4 * c);
                s[hh] = fmaf(k4.x, q4.x, s[hh]);
                s[hh] = fmaf(k4.y, q4.y, s[hh]);
                s[hh] = fmaf(k4.z, q4.z, s[hh]);
                s[hh] = fmaf(k4.w, q4.w, s[hh]);
            }
        }
        __syncwarp();   // the previous tile's readers of Ps are done
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
            float v = s[hh] + __shfl_xor_sync(0xffffffffu, s[hh], 16);
            v = (t < valid) ? v * p.sm_scale : -INFINITY;
            float tmax = v;
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, d));
            const float m_new = fmaxf(st.m[hh], tmax);
            const float alpha = exp2f((st.m[hh] - m_new) * kLog2e);
            const float pr = exp2f((v - m_new) * kLog2e);
            st.l[hh] = st.l[hh] * alpha + (hf == 0 ? pr : 0.f);
            st.lw[hh] = st.lw[hh] * alpha + ((hf == 0 && watch_base + t >= st.wlo && watch_base + t < st.whi) ? pr : 0.f);
            st.m[hh] = m_new;
#pragma unroll
            for (int i = 0; i < V; ++i) st.o[hh][i] *= alpha;
            if (hf == 0) Ps[hh * kPage + t] = pr;
        }
        __syncwarp();
        const float *vcol = reinterpret_cast<const float *>(Vs) + lane * V;
        for (int tt = 0; tt < valid; ++tt) {   // rows past `valid` are never touched
            float vv[V];
            if constexpr (V == 4) { float4 x = *reinterpret_cast<const float4 *>(vcol + tt * D); vv[0] = x.x; vv[1] = x.y; vv[2] = x.z; vv[3] = x.w; }
            else { float2 x = *reinterpret_cast<const float2 *>(vcol + tt * D); vv[0] = x.x; vv[1] = x.y; }
#pragma unroll
            for (int hh = 0; hh < GE; ++hh) {
                const float pr = Ps[hh * kPage + tt];
#pragma unroll
                for (int i = 0; i < V; ++i) st.o[hh][i] = fmaf(pr, vv[i], st.o[hh][i]);
            }
        }
    }

    __device__ static __forceinline__ void finish(State &st, float *So, float *Sm, float *Sl, int lane) {
        constexpr int PITCH = D + 4;
#pragma unroll
        for (int hh = 0; hh < GE; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) So[hh * PITCH + lane * V + i] = st.o[hh][i];
            float l = st.l[hh], lw = st.lw[hh];
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) {
                l += __shfl_xor_sync(0xffffffffu, l, d);
                lw += __shfl_xor_sync(0xffffffffu, lw, d);
            }
            if (lane == 0) { Sm[hh] = st.m[hh]; Sl[hh] = l; Sl[kHeadsPerItem + hh] = lw; }
        }
        // rows beyond GE are never read by a complete segment, but a piece copies all 8 rows
        for (int hh = GE; hh < kHeadsPerItem; ++hh) {
#pragma unroll
            for (int i = 0; i < V; ++i) So[hh * PITCH + lane * V + i] = 0.f;
            if (lane == 0) { Sm[hh] = -INFINITY; Sl[hh] = 0.f; Sl[kHeadsPerItem + hh] = 0.f; }
        }
    }
};

// ------------------------------------------------------------------------------------------------
// Append inside the attention launch (protocol step 3a; Fig. 3 step 2).  The tile that holds the new token has
// just landed in shared memory with whatever the cache held at the token's slot; the warp overwrites that row of
// K and of V with the new rows, so that the query attends to its own token, and -- one head group per KV head --
// writes the same bytes through to the cache.  Other head groups of the KV head fetch the tile on their own
// and patch their own copy, so nobody depends on when the write lands.
template <class Math>
__device__ __forceinline__ void append_row(const Params &p, uint8_t *Ks, uint8_t *Vs, int u, int sq, int slot, int page, int lane) {
    constexpr int RB = Math::kTileBytes / kPage;     // bytes of one token row
    constexpr int NCH = RB / 16;
    const int kvh = sq / p.hgroups;
    const bool writer = sq - kvh * p.hgroups == 0;
    const int64_t src_row = (static_cast<int64_t>(u) * p.Hkv + kvh) * RB;
    const int64_t dst_row = ((static_cast<int64_t>(page) * p.Hkv + kvh) * kPage + slot) * RB;
    for (int i = lane; i < 2 * NCH; i += 32) {
        const int which = i / NCH, c = i - which * NCH;
        const uint4 val = *reinterpret_cast<const uint4 *>((which ? p.v_new : p.k_new) + src_row + c * 16);
        *reinterpret_cast<uint4 *>((which ? Vs : Ks) + Math::chunk_offset(slot, c)) = val;
        if (writer) *reinterpret_cast<uint4 *>((which ? p.v_pool_w : p.k_pool_w) + dst_row + c * 16) = val;
    }
    fence_proxy_async();
    __syncwarp();
}

// ------------------------------------------------------------------------------------------------
// Where a warp stands in the flattened tile stream.  Tiles are ordered by user, then sequence
// (kv head x head group), then page; tile index = S * (tiles of earlier users) + sq * np + j.
struct Cursor {
    int u, sq, j;          // user, sequence of the user, page tile of the sequence
    int np, npp;           // tiles per sequence of this user; of which private
    int base0, base1;      // page-table offsets of the user
    int len0, len1;        // token counts of the user
    int idx_cur, idx_next; // this lane's page index of the current / next batch of 32 tiles
    int key;               // (partition << 24 | batch) that idx_cur holds, -1 = nothing
};

constexpr int kUserCache = 1024;   // users whose validated tile counts a CTA keeps in shared memory

// Tile counts of user u: from the CTA's cache when it holds them (a launch that loaded its plan has no cache:
// cache == nullptr), else recomputed from the inputs.
__device__ __forceinline__ void cached_tiles(const Params &p, const int2 *cache, int u, int &n0, int &n1) {
    if (cache != nullptr && u < kUserCache) {
        const int2 v = cache[u];
        n0 = v.x;
        n1 = v.y;
    } else {
        user_tiles(p, u, n0, n1);
    }
}

__device__ __forceinline__ void cursor_load_user(Cursor &c, const Params &p, const int2 *cache) {
    int n0, n1;
    cached_tiles(p, cache, c.u, n0, n1);
    c.npp = n0;
    c.np = n0 + n1;
    c.base0 = p.part[0].present ? p.part[0].indptr[c.u] : 0;
    c.base1 = p.part[1].present ? p.part[1].indptr[c.u] : 0;
    c.len0 = p.part[0].present ? p.part[0].lens[c.u] : 0;
    c.len1 = p.part[1].present ? p.part[1].lens[c.u] + (p.k_new != nullptr ? 1 : 0) : 0;
    c.key = -1;
}

__device__ __forceinline__ int cursor_fetch_batch(const Cursor &c, const Params &p, int part, int batch, int lane) {
    const int i = batch * 32 + lane;
    const int n = part ? c.np - c.npp : c.npp;
    if (i >= n) return -1;
    return part ? p.part[1].indices[c.base1 + i] : p.part[0].indices[c.base0 + i];
}

// Shared-memory carve-up behind the rings: mbarriers (8 B each), then the per-stage descriptors
// (three int4 each, so 16-byte aligned), then each warp's private extra area (16-byte aligned).
template <class Math>
__host__ __device__ constexpr size_t attn_desc_offset() {
    return (static_cast<size_t>(Math::kWarps) * Math::kStages * 8 + 15) / 16 * 16;
}
template <class Math>
__host__ __device__ constexpr size_t attn_extra_offset() {
    return attn_desc_offset<Math>() + static_cast<size_t>(Math::kWarps) * Math::kStages * 48;
}
template <class Math>
__host__ __device__ constexpr size_t attn_bnd_offset() {
    return attn_extra_offset<Math>() + static_cast<size_t>(Math::kWarps) * Math::kExtraBytes;
}
// dynamic shared memory for a grid of `grid` CTAs: rings, barriers, descriptors, extras, share boundaries
template <class Math>
__host__ __device__ constexpr size_t attn_smem_bytes(int grid = 148) {
    return 1024 + static_cast<size_t>(Math::kWarps) * Math::kStages * 2 * Math::kTileBytes + attn_bnd_offset<Math>() +
           (static_cast<size_t>(grid) * Math::kWarps + 1) * 4 + 16;
}

template <class Math>
__global__ void __launch_bounds__(Math::kWarps * 32, 1)
attn_kernel(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mk0,
            const __grid_constant__ CUtensorMap mv0, const __grid_constant__ CUtensorMap mk1,
            const __grid_constant__ CUtensorMap mv1) {
    constexpr int D = Math::D, NS = Math::kStages, TB = Math::kTileBytes, NT = Math::kWarps * 32;
    static_assert(TB % 1024 == 0, "swizzled tiles need 1024-byte aligned bases");
    static_assert(Math::kExtraBytes % 16 == 0, "per-warp extra area holds float4 data");
    static_assert(2 * TB >= (kHeadsPerItem * (D + 4) + 3 * kHeadsPerItem) * 4, "a stage must hold the epilogue staging");
    static_assert(attn_smem_bytes<Math>(kMaxGrid) + 16384 <= 227 * 1024, "ring does not fit shared memory");
    static_assert(Math::kWarps <= 16 && Math::kStages >= 2, "CTA shape");
    static_assert(2 * Math::kWarps * 32 >= kMaxGrid, "every thread looks after at most two entries of the rate table");
    extern __shared__ uint8_t smem_raw[];
    __shared__ int32_t chunk_pfx[NT + 1];
    __shared__ int32_t warp_tot[Math::kWarps];
    __shared__ float red_w[Math::kWarps], red_r[Math::kWarps];
    __shared__ int32_t red_ok[Math::kWarps];
    __shared__ int32_t sh_wq[kMaxGrid], sh_pc[kMaxGrid + 1];
    __shared__ int2 sh_np[kUserCache];
    __shared__ long long cta_clock0;
    __shared__ int32_t cta_exits;
    __shared__ int32_t sh_jump[Math::kWarps][4];   // (user, sequence, tile) at which each warp resumes after its trailing piece
    __shared__ int32_t sh_prev_smid;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gwarp = blockIdx.x * Math::kWarps + wid;
    uint8_t *ring = base + static_cast<size_t>(wid) * NS * 2 * TB;
    uint8_t *tail = base + static_cast<size_t>(Math::kWarps) * NS * 2 * TB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail) + wid * NS;
    int4 *descs = reinterpret_cast<int4 *>(tail + attn_desc_offset<Math>()) + wid * NS * 3;
    uint8_t *extra = tail + attn_extra_offset<Math>() + static_cast<size_t>(wid) * Math::kExtraBytes;

    griddep_launch_dependents();   // the next kernel on the stream may begin its own read-only preamble
    // the four tensor maps are needed a few microseconds from now: fetch them meanwhile (when no partition owns a
    // page they are never used and hold nothing)
    if (wid == 0 && lane < 4 && (p.part[0].num_pages > 0 || p.part[1].num_pages > 0))
        prefetch_tensormap(lane == 0 ? &mk0 : lane == 1 ? &mv0 : lane == 2 ? &mk1 : &mv1);
    uint32_t smid;
    asm("mov.u32 %0, %%smid;" : "=r"(smid));

    const int C = (p.B + NT - 1) / NT;
    const int G = gridDim.x;
    // launch N on a workspace writes third N % 3 and reads the one launch N-2 wrote: launch N-1 may still be running
    const float2 *rate_rd = p.rates + ((p.rate_sel + 1) % 3) * kMaxGrid;
    float2 *rate_wr = p.rates + (p.rate_sel % 3) * kMaxGrid;
    int32_t *bnd = reinterpret_cast<int32_t *>(tail + attn_bnd_offset<Math>());
    const bool loaded = p.plan_mode == PLAN_LOAD;
    const int2 *np_cache = loaded ? nullptr : sh_np;
    int64_t T64 = 0;
    int T = 0, A = 0;
    bool plan_ok = true;
    int rec = 0;               // PLAN_LOAD: lane k < 8 holds word k of this warp's start record
    if (threadIdx.x == 0) cta_exits = 0;

    if (!loaded) {
    // ---- plan: every CTA computes the same thing from the inputs alone -------------------------
    // Thread t sums the tiles of users [t*C, (t+1)*C); a block scan gives chunk prefixes.
    {
        // the rate table travels together with the lengths: its loads are issued first and used last, so that
        // the two round trips to memory overlap (G <= 2 NT)
        const int i0 = threadIdx.x, i1 = threadIdx.x + NT;
        float2 v0 = make_float2(0.f, 0.f), v1 = make_float2(0.f, 0.f);
        if (i0 < G) v0 = __ldcg(rate_rd + i0);
        if (i1 < G) v1 = __ldcg(rate_rd + i1);
        int sum = 0;
        const int ub = threadIdx.x * C, ue = min(p.B, ub + C);
        for (int u = ub; u < ue; ++u) {
            int n0, n1;
            user_tiles(p, u, n0, n1);
            if (u < kUserCache) sh_np[u] = make_int2(n0, n1);
            sum += n0 + n1;
        }
        // rate = weight / cycles of the entries this thread looks after; their sums over the table by one
        // fixed tree (butterfly inside a warp, warps in order), so that every thread of every CTA gets the same bits
        const float r0 = (v0.x > 0.f && v0.y > 0.f) ? v0.x / v0.y : 0.f, r1 = (v1.x > 0.f && v1.y > 0.f) ? v1.x / v1.y : 0.f;
        float sw = (i0 < G ? v0.x : 0.f) + (i1 < G ? v1.x : 0.f), sr = r0 + r1;
        const bool ok_mine = (i0 >= G || r0 > 0.f) && (i1 >= G || r1 > 0.f);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            sw += __shfl_xor_sync(0xffffffffu, sw, d);
            sr += __shfl_xor_sync(0xffffffffu, sr, d);
        }
        const bool ok_warp = __all_sync(0xffffffffu, ok_mine);
        if (lane == 0) { red_w[wid] = sw; red_r[wid] = sr; red_ok[wid] = ok_warp; }
        int inc = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += t;
        }
        if (lane == 31) warp_tot[wid] = inc;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < wid; ++w) before += warp_tot[w];
        chunk_pfx[threadIdx.x] = before + inc - sum;
        if (threadIdx.x == NT - 1) chunk_pfx[NT] = before + inc;
        // ---- shares, first half: CTAs do not all stream at the same rate (some SMs sit behind busier
        // ports), so shares are sized by the rates measured on an earlier call that used this workspace: each
        // CTA left its (weight, cycles) in the rate table.  New weight = old weight moved towards the measured
        // rate (both relative to the mean): most of the way when they disagree by more than 4 % (a real
        // difference between SMs), a quarter of the way otherwise (so that run-to-run noise is averaged out
        // instead of chased); quantised to integers so that all CTAs cut alike.  With p.uniform every CTA
        // weighs the same and the table is not consulted.
        float tw = 0.f, tr = 0.f;
        bool ok = p.uniform == 0;
        for (int w = 0; w < Math::kWarps; ++w) { tw += red_w[w]; tr += red_r[w]; ok = ok && red_ok[w] != 0; }
        const float nw = ok ? G / tw : 0.f, nr = ok ? G / tr : 0.f;
        auto quantise = [&](float w_old, float r) {
            const float wn = w_old * nw, rn = r * nr;
            const float gain = fabsf(rn - wn) > 0.04f * wn ? 0.75f : 0.25f;
            const float m = ok ? wn + gain * (rn - wn) : 1.f;
            const int q = static_cast<int>(m * 1024.f + 0.5f);
            return q < 512 ? 512 : (q > 2048 ? 2048 : q);
        };
        if (i0 < G) sh_wq[i0] = quantise(v0.x, r0);
        if (i1 < G) sh_wq[i1] = quantise(v1.x, r1);
        __syncthreads();
    }
    T64 = static_cast<int64_t>(chunk_pfx[NT]) * p.S;
    T = T64 >= (1ll << 31) ? 0 : static_cast<int>(T64);

    // ---- shares, second half: warp w of the grid owns tiles [bnd[w], bnd[w+1]); prefix sums of the CTA weights
    if (wid == 0) {
        const int cpl = (G + 31) / 32;      // lane l looks after CTAs [l*cpl, (l+1)*cpl)
        int mysum = 0;
        for (int i = lane * cpl; i < min(G, (lane + 1) * cpl); ++i) mysum += sh_wq[i];
        int inc = mysum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += t;
        }
        int acc = inc - mysum;
        for (int i = lane * cpl; i < min(G, (lane + 1) * cpl); ++i) { sh_pc[i] = acc; acc += sh_wq[i]; }
        if (lane == 31) sh_pc[G] = inc;
    }
    __syncthreads();
    {
        const int64_t want = (static_cast<int64_t>(T) + p.min_tiles - 1) / p.min_tiles;   // warps that get a share
        A = want > p.num_warps ? p.num_warps : static_cast<int>(want);
    }
    {
        auto wsum = [&](int w) {     // weights of warps < w; a CTA's warps all carry the CTA's weight
            const int c = w / Math::kWarps;
            return static_cast<int64_t>(Math::kWarps) * sh_pc[c] + static_cast<int64_t>(w - c * Math::kWarps) * (c < G ? sh_wq[c] : 0);
        };
        // T * wsum(w) / total in double: the product is an integer below 2^53, hence exact; the quotient may
        // land one tile off where it is within an ulp of an integer, which moves a cut by a tile and nothing else
        // (every CTA computes the same bits; wsum is monotone; w = A gives T exactly)
        const double total = A > 0 ? static_cast<double>(wsum(A)) : 1.0;
        for (int w = threadIdx.x; w <= A; w += NT)
            bnd[w] = static_cast<int32_t>(static_cast<double>(T) * static_cast<double>(wsum(w)) / total);
    }
    __syncthreads();
    } else {
    // ---- plan loaded: an earlier launch on this stream and workspace, over the same lengths, left its share
    // boundaries, the CTA weights and every warp's starting point in the workspace.  If that launch is the previous
    // kernel on the stream it has completed, and its writes are visible, once the wait below returns; an older one
    // had left every SM before this launch could start.
        if (!p.plan_early) griddep_wait();
        const int32_t *pl = p.plan;
        T = __ldcg(pl + PLAN_T);
        A = __ldcg(pl + PLAN_A);
        plan_ok = __ldcg(pl + PLAN_TAG) == p.plan_tag && __ldcg(pl + PLAN_GRID) == G &&
                  __ldcg(pl + PLAN_WARPS) == Math::kWarps && __ldcg(pl + PLAN_B) == p.B && __ldcg(pl + PLAN_S) == p.S &&
                  __ldcg(pl + PLAN_PARTS) == (p.part[0].present | (p.part[1].present << 1)) && T >= 0 && A >= 0 &&
                  A <= p.num_warps;
        if (!plan_ok) T = A = 0;     // nothing is streamed; the status says why
        T64 = T;
        for (int w = threadIdx.x; w <= A; w += NT) bnd[w] = __ldcg(pl + PLAN_BND + w);
        if (threadIdx.x == 0) sh_wq[blockIdx.x] = __ldcg(pl + PLAN_WQ + blockIdx.x);
        if (lane < 8 && gwarp < A) rec = __ldcg(pl + PLAN_REC + gwarp * 8 + lane);
        __syncthreads();
    }

    const int t0 = gwarp < A ? bnd[gwarp] : 0;
    const int n = gwarp < A ? bnd[gwarp + 1] - t0 : 0;
    const int t1 = t0 + n;
    int tb = t0;               // the warp streams [tb, t1) first, then [t0, tb)
    Cursor c;
    c.u = c.sq = c.j = 0;

    // Where tile t sits: its user (the u with S * pfx[u] <= t < S * pfx[u + 1]), the tiles per
    // sequence of that user, the sequence and the tile within it.  (Needs the derived plan.)
    auto seq_of_tile = [&](int t, int &u, int &np, int &sq, int &jt) {
        const int x = t / p.S;    // in units of tiles per sequence
        int lo = 0, hi = NT;      // invariant: chunk_pfx[lo] <= x < chunk_pfx[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (chunk_pfx[mid] <= x) lo = mid; else hi = mid;
        }
        int acc = chunk_pfx[lo], n0 = 0, n1 = 0;
        for (u = lo * C;; ++u) {  // ends inside the chunk, because the chunk holds tile x
            cached_tiles(p, sh_np, u, n0, n1);
            if (acc + n0 + n1 > x) break;
            acc += n0 + n1;
        }
        np = n0 + n1;
        const int r = t - acc * p.S;
        sq = r / np;
        jt = r - sq * np;
    };

    // Order of work.  A share usually ends inside a sequence; that trailing piece needs a ticket
    // (a fence and an atomic, perhaps a merge: round trips to memory).  Done last they would be
    // exposed at the end of the kernel, done first the other warps cover them.  So the warp
    // streams [tb, t1) -- its trailing piece -- first and [t0, tb) afterwards.  Where the warp starts
    // (tile tb) and where it resumes (tile t0, kept in shared memory until then) make up its start record.
    if (n > 0) {
        int ju = 0, jsq = 0, jj = 0;
        if (!loaded) {
            int u, np, sq, jt;
            seq_of_tile(t1 - 1, u, np, sq, jt);
            if (jt != np - 1 && t1 - 1 - jt > t0) tb = t1 - 1 - jt;
            seq_of_tile(tb, c.u, np, c.sq, c.j);
            if (tb != t0) seq_of_tile(t0, ju, np, jsq, jj);
        } else {
            tb = __shfl_sync(0xffffffffu, rec, 0);
            c.u = __shfl_sync(0xffffffffu, rec, 1);
            c.sq = __shfl_sync(0xffffffffu, rec, 2);
            c.j = __shfl_sync(0xffffffffu, rec, 3);
            ju = __shfl_sync(0xffffffffu, rec, 4);
            jsq = __shfl_sync(0xffffffffu, rec, 5);
            jj = __shfl_sync(0xffffffffu, rec, 6);
            if (tb < t0 || tb >= t1) tb = t0;      // cannot happen with a plan this kernel stored
        }
        if (lane == 0) { sh_jump[wid][0] = ju; sh_jump[wid][1] = jsq; sh_jump[wid][2] = jj; }
        rec = lane == 0 ? tb : lane == 1 ? c.u : lane == 2 ? c.sq : lane == 3 ? c.j : lane == 4 ? ju : lane == 5 ? jsq : jj;
        __syncwarp();
    }

    // Everything up to the first tile loads only READS the call's inputs (lengths, page tables, the
    // KV pools, a rate table nobody writes any more), so it may run while the previous kernel on the
    // stream is still finishing on other SMs.  What follows touches the workspace, q, an incoming
    // partial and the outputs, and waits for that kernel (griddep_wait below).
    auto after_previous_kernel = [&]() {
        griddep_wait();
        if (threadIdx.x == 0) {
            cta_clock0 = clock64();
            sh_prev_smid = __ldcg(p.plan + PLAN_SMID + blockIdx.x);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            p.hdr[HDR_BATCH] = p.B;
            p.hdr[HDR_NSEQ] = p.B * p.S;
            if (T64 >= (1ll << 31)) flag_error(p.hdr, 2 /* SPD_ERR_UNSUPPORTED */, -1);   // 32-bit tile counter
            if (!plan_ok) flag_error(p.hdr, 7 /* SPD_ERR_PLAN */, -1);
        }
        // the plan stays in the workspace: boundaries and weights always (for inspection), the start records and
        // a valid tag when a later launch is to load it
        if (!loaded) {
            int32_t *pl = p.plan;
            if (blockIdx.x == 0) {
                for (int w = threadIdx.x; w <= A; w += NT) pl[PLAN_BND + w] = bnd[w];
                for (int i = threadIdx.x; i < G; i += NT) pl[PLAN_WQ + i] = sh_wq[i];
                if (threadIdx.x == 0) {
                    pl[PLAN_TAG] = p.plan_mode == PLAN_DERIVE_STORE ? p.plan_tag : 0;
                    pl[PLAN_T] = T; pl[PLAN_A] = A; pl[PLAN_GRID] = G; pl[PLAN_WARPS] = Math::kWarps;
                    pl[PLAN_B] = p.B; pl[PLAN_S] = p.S;
                    pl[PLAN_PARTS] = p.part[0].present | (p.part[1].present << 1);
                }
            }
            if (p.plan_mode == PLAN_DERIVE_STORE && n > 0 && lane < 8) pl[PLAN_REC + gwarp * 8 + lane] = rec;
            __threadfence();
        }
        // users that own no tile (nothing cached, or tables inconsistent): written and flagged here
        if (plan_ok)
        for (int u = gwarp; u < p.B; u += p.num_warps) {
            int n0, n1;
            cached_tiles(p, np_cache, u, n0, n1);
            if (n0 + n1 != 0) continue;
            const bool bad = user_tiles<true>(p, u, n0, n1);
            for (int sq = 0; sq < p.S; ++sq) {
                const int hbase = first_head(p, sq);
                for (int hh = 0; hh < p.geff; ++hh) {
                    float o[D / 32];
#pragma unroll
                    for (int i = 0; i < D / 32; ++i) o[i] = 0.f;
                    finalize_store<D>(p, u, hbase + hh, o, -INFINITY, 0.f, lane, bad);
                }
            }
        }
    };
    if (n <= 0) after_previous_kernel();
    if (n > 0) {

    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&bars[s]), 1);
        fence_mbar_init();
    }
    __syncwarp();

    const int n2 = tb == t0 ? n : t1 - tb;   // tiles streamed before the jump back to t0
    cursor_load_user(c, p, np_cache);
    int cur_t = tb;            // index in the tile stream of the next tile to issue

    const uint64_t stream_policy = l2_evict_first_policy();
    int issued = 0;            // tiles handed to the TMA so far
    bool seg_from0 = false;    // the segment being issued began at the start of its sequence
    bool seg_has_t0 = false;   // ... and holds the share's first tile

    auto issue = [&](int stage) {
        if (issued == n2 && n2 < n) {      // the trailing piece is out: back to the share's first tile
            c.u = sh_jump[wid][0]; c.sq = sh_jump[wid][1]; c.j = sh_jump[wid][2];
            cursor_load_user(c, p, np_cache);
            cur_t = t0;
        }
        // page of tile (c.u, c.sq, c.j)
        const int part = c.j >= c.npp ? 1 : 0;
        const int jj = part ? c.j - c.npp : c.j;
        const int key = (part << 24) | (jj >> 5);
        if (key != c.key) {
            c.idx_cur = (c.key >= 0 && key == c.key + 1) ? c.idx_next : cursor_fetch_batch(c, p, part, jj >> 5, lane);
            c.idx_next = cursor_fetch_batch(c, p, part, (jj >> 5) + 1, lane);
            c.key = key;
        }
        const int page = __shfl_sync(0xffffffffu, c.idx_cur, jj & 31);
        const int npart = part ? c.np - c.npp : c.npp;
        int valid = kPage;
        if (jj == npart - 1) valid = (part ? c.len1 : c.len0) - jj * kPage;
        const bool first = (c.j == 0) || (cur_t == t0);
        const bool last = (c.j == c.np - 1) || (cur_t == t1 - 1);
        if (first) { seg_from0 = (c.j == 0); seg_has_t0 = (cur_t == t0); }
        int kind = 0;
        if (last && !(seg_from0 && c.j == c.np - 1)) kind = seg_has_t0 ? 1 : 2;
        if (page < 0 || page >= p.part[part].num_pages) valid = 0;   // never fetched; flagged when consumed
        const bool newtok = p.k_new != nullptr && part == 1 && jj == npart - 1;   // the tile that takes the appended row
        if (lane == 0) {
            descs[3 * stage] = make_int4(valid, (first ? 1 : 0) | (last ? 2 : 0) | (newtok ? 4 : 0) | (kind << 8), c.u, c.sq);
            descs[3 * stage + 1] = make_int4(c.np, c.j, cur_t, c.npp);
            descs[3 * stage + 2] = make_int4(page, 0, 0, 0);
            const uint32_t bar = smem_u32(&bars[stage]);
            if (valid == 0) {
                mbar_arrive(bar);
            } else {
                const int kvh = c.sq / p.hgroups;
                const int row = (page * p.Hkv + kvh) * kPage;
                const uint32_t kdst = smem_u32(ring + static_cast<size_t>(stage) * 2 * TB), vdst = kdst + TB;
                const CUtensorMap *mk = part ? &mk1 : &mk0, *mv = part ? &mv1 : &mv0;
                mbar_expect_tx(bar, 2 * TB);
#pragma unroll
                for (int b = 0; b < Math::kBoxes; ++b) {
                    tma_load_2d(kdst + b * Math::kBoxBytes, mk, b * Math::kBoxCols, row, bar, stream_policy);
                    tma_load_2d(vdst + b * Math::kBoxBytes, mv, b * Math::kBoxCols, row, bar, stream_policy);
                }
            }
        }
        ++issued;
        ++cur_t;
        // advance to the next tile (skipping users that own no tile), unless the range ends here
        if (issued != n && issued != n2 && ++c.j == c.np) {
            c.j = 0;
            if (++c.sq == p.S) {
                c.sq = 0;
                do {
                    if (c.u + 1 >= p.B) {     // only a loaded plan that no longer fits the lengths runs off the end
                        c.np = c.npp = 0;
                        if (lane == 0) flag_error(p.hdr, 7 /* SPD_ERR_PLAN */, -1);
                        break;
                    }
                    ++c.u;
                    cursor_load_user(c, p, np_cache);
                } while (c.np == 0);
            } else {
                c.key = -1;   // same user, page table starts over
            }
        }
    };

    for (int s = 0; s < NS && s < n; ++s) issue(s);
    after_previous_kernel();

    typename Math::State st;
    bool seg_bad = false, dead = false;
    int i = 0;
    for (; i < n; ++i) {
        const int stage = i % NS;
        if (!mbar_wait(smem_u32(&bars[stage]), (i / NS) & 1)) { dead = true; break; }
        const int4 d = descs[3 * stage];
        uint8_t *Ks = ring + static_cast<size_t>(stage) * 2 * TB, *Vs = Ks + TB;
        if (d.y & 1) { Math::begin(st, p, d.z, d.w, lane, extra); seg_bad = false; }
        const int4 e = descs[3 * stage + 1];
        if ((d.y & 4) && d.x > 0) append_row<Math>(p, Ks, Vs, d.z, d.w, d.x - 1, descs[3 * stage + 2].x, lane);
        if (d.x > 0) {
            Math::tile(st, p, Ks, Vs, d.x, lane, extra, e.y < e.w ? e.y * kPage : -(1 << 30));
        } else {                                   // a page index outside the pool: flag the user, skip the tile
            seg_bad = true;
            if (lane == 0) { p.bad[d.z] = p.epoch; flag_error(p.hdr, 4 /* SPD_ERR_BAD_PAGE */, d.z); }
        }
        if (d.y & 2) {
            // the stage just consumed doubles as the staging area of the epilogue
            __syncwarp();
            float *So = reinterpret_cast<float *>(Ks);
            float *Sm = So + kHeadsPerItem * (D + 4), *Sl = Sm + kHeadsPerItem;
            Math::finish(st, So, Sm, Sl, lane);
            __syncwarp();
            const int kind = d.y >> 8;
            if (kind == 0) {
                // a chained step's second half: a user flagged by the first half (same call id) stays zeroed
                const bool flagged = p.in_o != nullptr && __ldcg(p.bad + d.z) == p.epoch;
                finalize_segment<D>(p, So, Sm, Sl, d.z, d.w, lane, seg_bad || flagged);
            } else {
                piece_store<D>(p, So, Sm, Sl, kind, gwarp, lane);
                const PieceInfo pp{d.z, d.w, e.x, e.z - e.y, seg_bad};
                piece_ticket<D>(p, pp, bnd, A, lane);
            }
            fence_proxy_async();
        }
        __syncwarp();
        if (issued < n) issue(stage);
    }
    if (dead) {
        if (lane == 0) flag_error(p.hdr, 6 /* SPD_ERR_TIMEOUT */, -1);
        // give the copies still in flight a bounded chance to land before the warp leaves
        for (int k = i + 1; k < issued; ++k) mbar_wait(smem_u32(&bars[k % NS]), (k / NS) & 1);
    }

    }   // n > 0

    // ---- the CTA's last warp out leaves (weight, cycles) for the next call's shares -------------
    __syncwarp();
    __threadfence();      // this warp's flags and rows are visible before anybody can see it counted out
    int last_cta = 0;
    if (lane == 0 && atomicAdd(&cta_exits, 1) == Math::kWarps - 1) {
        const int wa = blockIdx.x * Math::kWarps, wb = wa + Math::kWarps;
        const int tiles = (wb <= A ? bnd[wb] : T) - (wa <= A ? bnd[wa] : T);
        float2 v = __ldcg(rate_rd + blockIdx.x);                   // a call too small to tell keeps the old entry
        if (tiles >= 32 * Math::kWarps)
            v = make_float2(static_cast<float>(sh_wq[blockIdx.x]), static_cast<float>(clock64() - cta_clock0));
        __stcg(rate_wr + blockIdx.x, v);
        // The rates belong to SMs, the table is indexed by CTA: count how often a CTA index comes back on another SM
        // than at the previous launch on this workspace (read by spd_debug_sm_moves).
        const int sm = static_cast<int>(smid) + 1, prev = sh_prev_smid;
        if (prev != 0) {
            if (prev != sm) atomicAdd(&p.hdr[HDR_SM_MOVES], 1);
            if (blockIdx.x == 0) atomicAdd(&p.hdr[HDR_SM_LAUNCHES], 1);
        }
        p.plan[PLAN_SMID + blockIdx.x] = sm;
        if (p.k_new != nullptr) {
            __threadfence();
            last_cta = atomicAdd(&p.hdr[HDR_GRID_EXITS], 1) == G - 1;
        }
    }
    if (p.k_new == nullptr) return;
    // ---- an appending launch: once every CTA has finished (nobody reads the lengths any more), the last warp out
    // of the last CTA makes the new token count: length + 1 for every user that this call did not flag
    last_cta = __shfl_sync(0xffffffffu, last_cta, 0);
    if (!last_cta) return;
    if (lane == 0) p.hdr[HDR_GRID_EXITS] = 0;
    __threadfence();
    for (int base = 0; base < p.B; base += 256) {
        int32_t fl[8], ln[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int u = base + k * 32 + lane;
            fl[k] = u < p.B ? __ldcg(p.bad + u) : p.epoch;
            ln[k] = u < p.B ? __ldcg(p.lens_w + u) : 0;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int u = base + k * 32 + lane;
            if (u < p.B && fl[k] != p.epoch) p.lens_w[u] = ln[k] + 1;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Append of the new token's K and V rows to a paged cache (protocol step 3a; Fig. 3 step 2): one CTA
// per user.  The row of user u goes to token position len_u -- page indices[indptr[u] + len_u / 16],
// slot len_u % 16 -- and len_u grows by one.  A user whose listed pages are full, or whose table is
// inconsistent, is left untouched and flagged.  Plain 16-byte copies: a few hundred KB per call.
struct AppendParams {
    int32_t B, Hkv, row_bytes;      // row_bytes = head_dim * element size
    const uint8_t *k_new, *v_new;   // [B][Hkv][row_bytes]
    uint8_t *k_pool, *v_pool;
    int32_t num_pages;
    const int32_t *indptr, *indices;
    int32_t *lens;
    int32_t *hdr;
};

__global__ void __launch_bounds__(128) append_kernel(AppendParams p) {
    const int u = blockIdx.x;
    __shared__ int64_t dst_row;   // byte offset of (page, kv head 0, slot) in a pool, or -1
    if (threadIdx.x == 0) {
        const int64_t lo = p.indptr[u], hi = p.indptr[u + 1], end = p.indptr[p.B], t = p.lens[u];
        int64_t off = -1;
        if (lo >= 0 && hi >= lo && hi <= end && t >= 0 && t < (hi - lo) * kPage && p.indices != nullptr) {
            const int64_t page = p.indices[lo + t / kPage];
            if (page >= 0 && page < p.num_pages) off = ((page * p.Hkv) * kPage + t % kPage) * p.row_bytes;
        }
        if (off < 0) flag_error(p.hdr, 4 /* SPD_ERR_BAD_PAGE */, u);
        dst_row = off;
    }
    __syncthreads();
    const int64_t off = dst_row;
    if (off < 0) return;
    const int chunks = p.row_bytes / 16, total = p.Hkv * chunks;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int h = i / chunks, c = i - h * chunks;
        const int64_t src = (static_cast<int64_t>(u) * p.Hkv + h) * p.row_bytes + c * 16;
        const int64_t dst = off + static_cast<int64_t>(h) * kPage * p.row_bytes + c * 16;
        *reinterpret_cast<uint4 *>(p.k_pool + dst) = *reinterpret_cast<const uint4 *>(p.k_new + src);
        *reinterpret_cast<uint4 *>(p.v_pool + dst) = *reinterpret_cast<const uint4 *>(p.v_new + src);
    }
    __syncthreads();
    if (threadIdx.x == 0) p.lens[u] += 1;
}

// ------------------------------------------------------------------------------------------------
// Merge of up to kMaxMergeParts partials into the normalised attention output (Theorem 1 / Eq. 1 with
// the maxima of Sec. 4.2, n-way): one warp per (user, query head), lane = D/32 channels.
constexpr int kMaxMergeParts = 8;
struct MergeParams {
    int32_t rows, n, out_bf16;     // rows = batch * num_q_heads
    const float *o[kMaxMergeParts], *m[kMaxMergeParts], *l[kMaxMergeParts];
    void *out;
};

template <int D>
__global__ void __launch_bounds__(128) merge_partials_kernel(MergeParams p) {
    constexpr int V = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
    if (row >= p.rows) return;
    float M = -INFINITY;
    for (int c = 0; c < p.n; ++c) M = fmaxf(M, p.m[c][row]);
    float L = 0.f, o[V];
#pragma unroll
    for (int i = 0; i < V; ++i) o[i] = 0.f;
    for (int c = 0; c < p.n; ++c) {
        const float mc = p.m[c][row];
        const float w = (mc == -INFINITY) ? 0.f : expf(mc - M);
        L = fmaf(w, p.l[c][row], L);
        const float *src = p.o[c] + row * D + lane * V;
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = fmaf(w, src[i], o[i]);
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) o[i] = inv == 0.f ? 0.f : o[i] * inv;
    if (p.out_bf16) {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + row * D + lane * V;
#pragma unroll
        for (int i = 0; i < V; i += 2) *reinterpret_cast<__nv_bfloat162 *>(dst + i) = __floats2bfloat162_rn(o[i], o[i + 1]);
    } else {
        float *dst = reinterpret_cast<float *>(p.out) + row * D + lane * V;
#pragma unroll
        for (int i = 0; i < V; ++i) dst[i] = o[i];
    }
}

}  // namespace spd
