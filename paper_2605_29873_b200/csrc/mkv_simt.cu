// Scalar (fp32 FMA) split-KV decode attention: every dtype and head_dim the library
// accepts.  It is the path for fp32 caches (where tensor cores would cost precision) and
// the second, independent GPU implementation the tensor-core kernel is checked against.
//
// One CTA per item, four warps.  A warp owns whole cache rows: lane l holds head_dim/32
// consecutive elements of the row, so a row is one coalesced 128/256/512-byte access; the
// G query heads of the KV group share every K and V row (GQA).  Per row: G dot products
// (Eq. 2 logits, already in log2 units), a butterfly warp reduction, an online-softmax
// update of (m, l, O).  Warps are merged in shared memory, the CTA writes one partial and
// takes a ticket; the last ticket holder of the unit runs the tail.
#include "mkv_launch.h"
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

template <int BPL>
__device__ inline void copy_piece(uint8_t* dst, const uint8_t* src) {
    if constexpr (BPL == 16) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    else if constexpr (BPL == 8) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
    else *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
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
    const int4 it4 = *reinterpret_cast<const int4*>(&L.items[blockIdx.x]);
    const int u = it4.x, row0 = it4.y, rows = it4.z, seg = it4.w;
    const int b = u / p.kv_heads, g = u - b * p.kv_heads;
    const bool dec = (p.mode == kModeDecode);
    int n_old = L.n_dec[u];
    if (n_old + (dec ? 1 : 0) > p.cap) {   // cannot happen while budget <= cap - 1
        if (tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
        n_old = p.cap - (dec ? 1 : 0);
    }

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
    float* lg = L.logit + ((size_t)b * p.q_heads + (size_t)g * G) * p.cap;

    auto row_math = [&](const float (&kf)[EPL], const float (&vf)[EPL], int slot, bool store) {
        float s[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float a = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) a = fmaf(qf[h][e], kf[e], a);
            s[h] = a;
        }
#pragma unroll
        for (int off = 16; off; off >>= 1)
#pragma unroll
            for (int h = 0; h < G; ++h) s[h] += __shfl_xor_sync(0xffffffffu, s[h], off);
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if (store && lane == h) lg[(size_t)h * p.cap + slot] = s[h];
            const float mn = fmaxf(m[h], s[h]);
            const float sc = fast_exp2(m[h] - mn);
            const float pr = fast_exp2(s[h] - mn);
            l[h] = fmaf(l[h], sc, pr);
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(o[h][e], sc, pr * vf[e]);
            m[h] = mn;
        }
    };

    const uint8_t* kbase;
    const uint8_t* vbase;
    int valid_end;
    if (seg == 0) {
        kbase = L.Kp + (size_t)u * p.max_prefill * ROWB;
        vbase = L.Vp + (size_t)u * p.max_prefill * ROWB;
        valid_end = L.unit_lp[u];
    } else {
        kbase = L.Kd + (size_t)u * p.cap * ROWB;
        vbase = L.Vd + (size_t)u * p.cap * ROWB;
        valid_end = n_old;
    }
    const int r_end = min(row0 + rows, valid_end);
    const bool store = dec && seg == 1;
    for (int r = row0 + warp; r < r_end; r += kSimtWarps) {
        float kf[EPL], vf[EPL];
        const uint32_t off = swz((uint32_t)r, (uint32_t)(lane * BPL));
        load_piece<T, EPL>(kbase + (size_t)r * ROWB + off, kf);
        load_piece<T, EPL>(vbase + (size_t)r * ROWB + off, vf);
        row_math(kf, vf, r, store);
    }
    // Algorithm 1 append: the item whose range holds slot n_old takes the fresh token from
    // k_new / v_new, scores it like any other row and stores it into the pool.
    if (dec && seg == 1 && n_old >= row0 && n_old < row0 + rows && warp == 0) {
        const uint8_t* ks = reinterpret_cast<const uint8_t*>(p.k_new) + (size_t)u * ROWB + lane * BPL;
        const uint8_t* vs = reinterpret_cast<const uint8_t*>(p.v_new) + (size_t)u * ROWB + lane * BPL;
        float kf[EPL], vf[EPL];
        load_piece<T, EPL>(ks, kf);
        load_piece<T, EPL>(vs, vf);
        const uint32_t off = swz((uint32_t)n_old, (uint32_t)(lane * BPL));
        copy_piece<BPL>(L.Kd + ((size_t)u * p.cap + n_old) * ROWB + off, ks);
        copy_piece<BPL>(L.Vd + ((size_t)u * p.cap + n_old) * ROWB + off, vs);
        row_math(kf, vf, n_old, true);
    }

    // merge the four warps, write the partial
    if (lane == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h) { xm[warp][h] = m[h]; xl[warp][h] = l[h]; }
    }
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
        for (int e = 0; e < EPL; ++e) xo[warp][h][lane * EPL + e] = o[h][e];
    __syncthreads();
    const size_t part = blockIdx.x;
    for (int idx = tid; idx < G * D; idx += kSimtThreads) {
        const int h = idx / D, i = idx - h * D;
        float M = xm[0][h];
#pragma unroll
        for (int w = 1; w < kSimtWarps; ++w) M = fmaxf(M, xm[w][h]);
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < kSimtWarps; ++w) {
            const float sc = fast_exp2(xm[w][h] - M);
            acc = fmaf(xo[w][h][i], sc, acc);
            ls = fmaf(xl[w][h], sc, ls);
        }
        L.part_o[part * G * D + idx] = acc;
        if (i == 0) {
            L.part_ml[(part * G + h) * 2] = M;
            L.part_ml[(part * G + h) * 2 + 1] = ls;
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(&L.ticket[u], 1);
        s_last = (prev == L.unit_nparts[u] - 1);
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        unit_tail<kSimtThreads, 1>(p, u, tsm, tid, ROWB);
    }
    __syncthreads();
    if (tid == 0) grid_epilogue(p, gridDim.x);
}

template <typename T, int D>
cudaError_t launch_td(const Params& p, cudaStream_t st) {
    const dim3 grid((unsigned)p.L.n_items), block(kSimtThreads);
    switch (p.group) {
#define MKV_CASE(GG) case GG: simt_kernel<T, D, GG><<<grid, block, 0, st>>>(p); break;
        MKV_CASE(1) MKV_CASE(2) MKV_CASE(3) MKV_CASE(4) MKV_CASE(5) MKV_CASE(6) MKV_CASE(7) MKV_CASE(8)
#undef MKV_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

bool simt_supported(int kv_dtype, int head_dim, int group) {
    return (kv_dtype == 0 || kv_dtype == 1) && (head_dim == 64 || head_dim == 128) && group >= 1 && group <= 8;
}

cudaError_t launch_simt(const Params& p, int kv_dtype, cudaStream_t st) {
    if (p.L.n_items <= 0) return cudaSuccess;
    if (kv_dtype == 0) {
        return p.head_dim == 128 ? launch_td<__nv_bfloat16, 128>(p, st) : launch_td<__nv_bfloat16, 64>(p, st);
    }
    return p.head_dim == 128 ? launch_td<float, 128>(p, st) : launch_td<float, 64>(p, st);
}

}  // namespace mkv
