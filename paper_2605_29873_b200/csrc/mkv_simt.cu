// Scalar (fp32 FMA) split-KV decode attention: every dtype and head_dim the library
// accepts.  It is the path for fp32 caches (where tensor cores would cost precision) and
// the second, independent GPU implementation the tensor-core kernel is checked against.
//
// Persistent CTAs of four warps pull chunks of tiles from the per-unit counters, starting at
// their own place and moving on to the next unit with tiles left.  A warp owns whole
// cache rows: lane l holds head_dim/32 consecutive elements of the row, so a row is one
// coalesced 128/256/512-byte access; the G query heads of the KV group share every K and V
// row (GQA).  Per row: G dot products (Eq. 2 logits, already in log2 units), a butterfly
// warp reduction, an online-softmax update of (m, l, O).  At the end of a unit visit the warps
// are merged in shared memory and the CTA writes one partial with its tile count; the
// delivery that completes the unit runs its tail.  In the reproducible mode there are no
// counters: every CTA covers a fixed range of the global tile sequence and its partial of a
// unit goes to a fixed slot.
#include "mkv_launch.h"
#include "mkv_layer_tail.cuh"
#include "mkv_tail.cuh"

namespace mkv {
namespace {

constexpr int kSimtWarps = 4;
constexpr int kSimtThreads = kSimtWarps * 32;

template <typename T, int EPL>
__device__ inline void load_piece(const uint8_t* ptr, float (&f)[EPL]) {
    constexpr int BPL = EPL * (int)sizeof(T);
    if constexpr (BPL == 16) {
        const uint4 v = *reinterpret_cast<const uint4*>(ptr);
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < EPL; ++i) f[i] = to_f32(e[i]);
    } else if constexpr (BPL == 8) {
        const uint2 v = *reinterpret_cast<const uint2*>(ptr);
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < EPL; ++i) f[i] = to_f32(e[i]);
    } else {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(ptr);
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < EPL; ++i) f[i] = to_f32(e[i]);
    }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kSimtThreads) simt_kernel(const Params p) {
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int EPL = D / 32;
    constexpr int BPL = EPL * (int)sizeof(T);
    __shared__ TailSmem<kSimtThreads> tsm;
    __shared__ float xm[kSimtWarps][G], xl[kSimtWarps][G];
    __shared__ float xo[kSimtWarps][G][D];
    __shared__ int s_last;

    const LayerDev& L = p.L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool dec = (p.mode == kModeDecode);
    const int U = L.n_units;
    __shared__ int s_g, s_u;

    // which copy of the unit counters this launch uses
    if (tid == 0) tsm.par = take_launch_parity(L);
    __syncthreads();
    int32_t* const nxt = L.next + (size_t)tsm.par * L.n_units;
    int2* const cnt = L.cnt + (size_t)tsm.par * L.n_units;

    int u = L.cta_unit0[blockIdx.x];
    int head = L.cta_head0[blockIdx.x], headn = L.cta_headn[blockIdx.x];   // reserved tiles, first visit only
    const bool det = p.det != 0;
    int det_t = det ? L.cta_t0[blockIdx.x] : 0;                 // reproducible mode: next global tile ...
    const int det_end = det ? L.cta_t0[blockIdx.x + 1] : 0;     // ... and the end of this CTA's range
    for (;;) {
        if (det && det_t >= det_end) break;
        // ---- one visit of unit u: pull chunks until the unit has none left -------------------
        const int b = u / p.kv_heads, g = u - b * p.kv_heads;
        const int lp = L.unit_lp[u];
        int n_old = L.n_dec[u];
        if (n_old > p.cap - (dec ? 1 : 0)) {   // cannot happen while budget <= cap - 1
            if (tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
            n_old = p.cap - (dec ? 1 : 0);
        }
        const int chunk = L.unit_chunk[u];
        const int total = det ? L.tile_begin[u + 1] - L.tile_begin[u] : unit_tiles(lp, n_old);
        bool det_taken = false;
        float qf[G][EPL];
        {
            const T* qp = reinterpret_cast<const T*>(p.q) + ((size_t)b * p.q_heads + (size_t)g * G) * D + lane * EPL;
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < EPL; ++e) qf[h][e] = to_f32(qp[(size_t)h * D + e]) * p.scale_log2;
        }
        float m[G], l[G], o[G][EPL];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m[h] = kNegBig; l[h] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[h][e] = 0.f;
        }
        float* lg = L.logit + ((size_t)b * p.q_heads + (size_t)g * G) * p.lstride;
        int mine = 0;
        for (;;) {
            int t0, t1;
            if (det) {
                if (det_taken) break;
                det_taken = true;
                t0 = det_t - L.tile_begin[u];
                t1 = min(det_end, L.tile_begin[u + 1]) - L.tile_begin[u];
                det_t = L.tile_begin[u] + t1;
            } else if (headn > 0) { t0 = head; t1 = head + headn; headn = 0; }
            else {
                if (tid == 0) s_g = atomicAdd(&nxt[u], chunk);
                __syncthreads();
                t0 = s_g;
                __syncthreads();
                if (t0 >= total) break;
                t1 = min(t0 + chunk, total);
            }
            mine += t1 - t0;
            for (int t = t0; t < t1; ++t) {
                const TileRef tr = tile_ref(t, lp, n_old);
                const uint8_t* kbase = (tr.seg == 0 ? L.Kp + (size_t)u * p.max_prefill * ROWB : L.Kd + (size_t)u * p.cap * ROWB);
                const uint8_t* vbase = (tr.seg == 0 ? L.Vp + (size_t)u * p.max_prefill * ROWB : L.Vd + (size_t)u * p.cap * ROWB);
                const bool store = dec && tr.seg == 1;
                for (int r = tr.row + warp; r < tr.row + tr.cnt; r += kSimtWarps) {
                    float kf[EPL], vf[EPL];
                    const uint32_t off = swz((uint32_t)r, (uint32_t)(lane * BPL));
                    load_piece<T, EPL>(kbase + (size_t)r * ROWB + off, kf);
                    load_piece<T, EPL>(vbase + (size_t)r * ROWB + off, vf);
                    float sc[G];
#pragma unroll
                    for (int h = 0; h < G; ++h) {
                        float a = 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) a = fmaf(qf[h][e], kf[e], a);
                        sc[h] = a;
                    }
#pragma unroll
                    for (int off2 = 16; off2; off2 >>= 1)
#pragma unroll
                        for (int h = 0; h < G; ++h) sc[h] += __shfl_xor_sync(0xffffffffu, sc[h], off2);
#pragma unroll
                    for (int h = 0; h < G; ++h) {
                        if (store && lane == h) lg[(size_t)h * p.lstride + r] = sc[h];
                        const float mn = fmaxf(m[h], sc[h]);
                        const float fs = fast_exp2(m[h] - mn);
                        const float pr = fast_exp2(sc[h] - mn);
                        l[h] = fmaf(l[h], fs, pr);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(o[h][e], fs, pr * vf[e]);
                        m[h] = mn;
                    }
                }
            }
        }
        if (mine > 0) {
            // merge the four warps, write the visit's partial into a fresh slot of the unit
            if (tid == 0) {
                s_g = atomicAdd(&cnt[u].y, 1);
                if (det) s_g = (int)blockIdx.x - L.unit_cta0[u];    // a fixed slot: this CTA's rank in the unit
            }
            if (lane == 0) {
#pragma unroll
                for (int h = 0; h < G; ++h) { xm[warp][h] = m[h]; xl[warp][h] = l[h]; }
            }
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < EPL; ++e) xo[warp][h][lane * EPL + e] = o[h][e];
            __syncthreads();
            if (s_g >= kMaxParts && tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
            const size_t part = (size_t)u * kMaxParts + (size_t)min(s_g, kMaxParts - 1);
            for (int idx = tid; idx < G * D; idx += kSimtThreads) {
                const int h = idx / D, i = idx - h * D;
                float M = xm[0][h];
#pragma unroll
                for (int w = 1; w < kSimtWarps; ++w) M = fmaxf(M, xm[w][h]);
                float acc = 0.f, ls = 0.f;
#pragma unroll
                for (int w = 0; w < kSimtWarps; ++w) {
                    const float fs = fast_exp2(xm[w][h] - M);
                    acc = fmaf(xo[w][h][i], fs, acc);
                    ls = fmaf(xl[w][h], fs, ls);
                }
                L.part_o[part * G * D + idx] = acc;
                if (i == 0) {
                    L.part_ml[(part * G + h) * 2] = M;
                    L.part_ml[(part * G + h) * 2 + 1] = ls;
                }
            }
            __threadfence();
            __syncthreads();
            // the delivery that completes the unit's tile count runs its tail
            if (tid == 0) s_last = (atomicAdd(&cnt[u].x, mine) + mine == total);
            __syncthreads();
            if (s_last) {
                __threadfence();
                constexpr int GB = G <= 4 ? 4 : 8;
                TailPre<kSimtThreads, GB> pre;
                if (p.layer_mean) {
                    tail_prefetch<T, kSimtThreads, GB, true>(p, u, tsm, tid, pre);
                    layer_unit_tail<T, kSimtThreads, 1, GB>(p, u, __ldcg(&cnt[u].y), pre, tsm, tid);
                } else {
                    tail_prefetch<T, kSimtThreads, GB>(p, u, tsm, tid, pre);
                    unit_tail<T, kSimtThreads, 1, GB>(p, u, __ldcg(&cnt[u].y), pre, tsm, tid);
                }
            }
            __syncthreads();
        }
        // ---- next unit (cyclically after this one) that still has tiles to hand out -----------
        if (det) { ++u; if (u >= U) break; continue; }
        if (warp == 0) {     // 32 candidates per trip, the nearest one with tiles left wins
            int found = -1;
            for (int base = 1; base < U && base <= kHopWindow && found < 0; base += 32) {
                const int k = base + lane;
                bool has = false;
                if (k < U) {
                    const int cand = (u + k) % U;
                    const int nd = min(L.n_dec[cand], p.cap - (dec ? 1 : 0));
                    has = __ldcg(&nxt[cand]) < unit_tiles(L.unit_lp[cand], nd);
                }
                const unsigned m = __ballot_sync(0xffffffffu, has);
                if (m) found = (u + base + __ffs(m) - 1) % U;
            }
            if (lane == 0) s_u = found;
        }
        __syncthreads();
        u = s_u;
        __syncthreads();
        if (u < 0) break;
    }
}

template <typename T, int D>
cudaError_t launch_td(const Params& p, cudaStream_t st) {
    const dim3 grid((unsigned)p.L.n_ctas), block(kSimtThreads);
    switch (p.group) {
#define MKV_CASE(GG) case GG: simt_kernel<T, D, GG><<<grid, block, 0, st>>>(p); break;
        MKV_CASE(1) MKV_CASE(2) MKV_CASE(3) MKV_CASE(4) MKV_CASE(5) MKV_CASE(6) MKV_CASE(7) MKV_CASE(8)
#undef MKV_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t occupancy_td(int group, int* n) {
    switch (group) {
#define MKV_CASE(GG) case GG: return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, simt_kernel<T, D, GG>, kSimtThreads, 0);
        MKV_CASE(1) MKV_CASE(2) MKV_CASE(3) MKV_CASE(4) MKV_CASE(5) MKV_CASE(6) MKV_CASE(7) MKV_CASE(8)
#undef MKV_CASE
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t simt_occupancy(int kv_dtype, int head_dim, int group, int* resident_per_sm) {
    if (kv_dtype == 0)
        return head_dim == 128 ? occupancy_td<__nv_bfloat16, 128>(group, resident_per_sm)
                               : occupancy_td<__nv_bfloat16, 64>(group, resident_per_sm);
    return head_dim == 128 ? occupancy_td<float, 128>(group, resident_per_sm)
                           : occupancy_td<float, 64>(group, resident_per_sm);
}

bool simt_supported(int kv_dtype, int head_dim, int group) {
    return (kv_dtype == 0 || kv_dtype == 1) && (head_dim == 64 || head_dim == 128) && group >= 1 && group <= kMaxGroup;
}

cudaError_t launch_simt(const Params& p, int kv_dtype, cudaStream_t st) {
    if (p.L.n_ctas <= 0) return cudaSuccess;
    if (kv_dtype == 0) {
        return p.head_dim == 128 ? launch_td<__nv_bfloat16, 128>(p, st) : launch_td<__nv_bfloat16, 64>(p, st);
    }
    return p.head_dim == 128 ? launch_td<float, 128>(p, st) : launch_td<float, 64>(p, st);
}

}  // namespace mkv
