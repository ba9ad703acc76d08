// mkv_attend_noalloc: plain decode attention (Eq. 2) for callers that cannot allocate.
//
// Every other entry point of this library works inside a workspace the caller allocated.
// Some callers have no allocator to ask: code that runs after an inference server has
// handed all device memory to its own pool, plug-ins that are only given input and output
// buffers, or hosts where allocation is forbidden once serving has started.  For them this
// one call needs nothing but its inputs and outputs.  The split-KV partials and the tickets
// it needs between its CTAs live in a fixed array that is part of the library image, so
// every GPU that loads the library holds those few megabytes until the process exits, and
// problem sizes are capped by the array's size.
//
// The array is shared by all calls.  It keeps whatever the previous call left behind: the
// tickets are cleared at the start of every call and the partials are fully overwritten
// before they are read.  Two calls whose kernels overlap on the GPU (different streams)
// would use the same scratch at the same time and corrupt each other; callers must order
// them.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mkv.h"

namespace {

constexpr int kNaChunkRows = 256;                  // cached tokens per split
constexpr int kNaMaxPartRows = MKV_NOALLOC_MAX_PART_ROWS;   // batch * q_heads * splits
constexpr int kNaMaxUnits = MKV_NOALLOC_MAX_UNITS;          // batch * kv_heads
constexpr int kNaPartStride = 132;                 // floats per partial row: O[<=128], m, l, pad
constexpr int kNaThreads = 128;
constexpr int kNaMaxDevices = 64;
constexpr float kNaNegBig = -1.0e30f;

// [partial rows][132] floats, then [units] tickets
static __device__ __align__(256) float g_na_scratch[(size_t)kNaMaxPartRows * kNaPartStride + kNaMaxUnits];

__device__ inline float na_f32(float x) { return x; }
__device__ inline float na_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ inline float na_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct NaParams {
    const void *q, *K, *V;
    void* out;
    float* parts;      // device address of the static scratch
    int* tickets;
    int batch, q_heads, kv_heads, group, n_tokens, kv_rows, splits;
    float scale_log2;
    int out_f32;
};

// grid (splits, units).  A warp owns whole rows; lane l holds D/32 consecutive elements.
template <typename T, int D>
__global__ void __launch_bounds__(kNaThreads) na_attend_kernel(const NaParams p) {
    constexpr int EPL = D / 32;
    constexpr int GB = 8;
    __shared__ float xm[4][GB], xl[4][GB];
    __shared__ float xo[4][GB][D];
    __shared__ float cw[64][GB];
    __shared__ float cM[GB], cInvL[GB];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, u = blockIdx.y;
    const int b = u / p.kv_heads, g = u - b * p.kv_heads;
    const int G = p.group;
    const T* qp = reinterpret_cast<const T*>(p.q) + ((size_t)b * p.q_heads + (size_t)g * G) * D + lane * EPL;
    const T* kp = reinterpret_cast<const T*>(p.K) + (size_t)u * p.kv_rows * D + lane * EPL;
    const T* vp = reinterpret_cast<const T*>(p.V) + (size_t)u * p.kv_rows * D + lane * EPL;

    float qf[GB][EPL], m[GB], l[GB], o[GB][EPL];
#pragma unroll
    for (int h = 0; h < GB; ++h) {
        m[h] = kNaNegBig; l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            o[h][e] = 0.f;
            qf[h][e] = h < G ? na_f32(qp[(size_t)h * D + e]) * p.scale_log2 : 0.f;
        }
    }
    const int r0 = split * kNaChunkRows, r1 = min(r0 + kNaChunkRows, p.n_tokens);
    for (int r = r0 + warp; r < r1; r += 4) {
        float kf[EPL], vf[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) { kf[e] = na_f32(kp[(size_t)r * D + e]); vf[e] = na_f32(vp[(size_t)r * D + e]); }
#pragma unroll
        for (int h = 0; h < GB; ++h) {
            if (h < G) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(qf[h][e], kf[e], s);
#pragma unroll
                for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                const float mn = fmaxf(m[h], s);
                const float sc = na_exp2(m[h] - mn), pr = na_exp2(s - mn);
                l[h] = fmaf(l[h], sc, pr);
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(o[h][e], sc, pr * vf[e]);
                m[h] = mn;
            }
        }
    }
    // merge the four warps into one partial row per head
#pragma unroll
    for (int h = 0; h < GB; ++h) {
        if (h < G) {
            if (lane == 0) { xm[warp][h] = m[h]; xl[warp][h] = l[h]; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) xo[warp][h][lane * EPL + e] = o[h][e];
        }
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += kNaThreads) {
        const int h = idx / D, i = idx - h * D;
        float M = fmaxf(fmaxf(xm[0][h], xm[1][h]), fmaxf(xm[2][h], xm[3][h]));
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float sc = na_exp2(xm[w][h] - M);
            acc = fmaf(xo[w][h][i], sc, acc);
            ls = fmaf(xl[w][h], sc, ls);
        }
        float* row = p.parts + ((size_t)(u * G + h) * p.splits + split) * kNaPartStride;
        row[i] = acc;
        if (i == 0) { row[128] = M; row[129] = ls; }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&p.tickets[u], 1) == p.splits - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // last CTA of the unit: cross-split log-sum-exp combine
    const float* base = p.parts + (size_t)u * G * p.splits * kNaPartStride;
    if (tid < G) {
        float M = kNaNegBig;
        for (int s = 0; s < p.splits; ++s) M = fmaxf(M, __ldcg(base + ((size_t)tid * p.splits + s) * kNaPartStride + 128));
        float L = 0.f;
        for (int s = 0; s < p.splits; ++s) {
            const float* row = base + ((size_t)tid * p.splits + s) * kNaPartStride;
            const float w = na_exp2(__ldcg(row + 128) - M);
            cw[s][tid] = w;
            L = fmaf(__ldcg(row + 129), w, L);
        }
        cM[tid] = M;
        cInvL[tid] = L > 0.f ? 1.0f / L : 0.f;
    }
    __syncthreads();
    const size_t obase = ((size_t)b * p.q_heads + (size_t)g * G) * D;
    for (int idx = tid; idx < G * D; idx += kNaThreads) {
        const int h = idx / D, i = idx - h * D;
        float acc = 0.f;
        for (int s = 0; s < p.splits; ++s)
            acc = fmaf(__ldcg(base + ((size_t)h * p.splits + s) * kNaPartStride + i), cw[s][h], acc);
        acc *= cInvL[h];
        if (p.out_f32) reinterpret_cast<float*>(p.out)[obase + idx] = acc;
        else reinterpret_cast<__nv_bfloat16*>(p.out)[obase + idx] = __float2bfloat16_rn(acc);
    }
    if (tid == 0) p.tickets[u] = 0;
}

float* g_na_ptr[kNaMaxDevices];   // device address of g_na_scratch, per device (0 = not set up)

}  // namespace

extern "C" mkv_status mkv_attend_noalloc(const void* q, const void* K, const void* V, void* out, int batch,
                                         int q_heads, int kv_heads, int head_dim, int n_tokens, int kv_rows,
                                         int kv_dtype, int out_dtype, int device, void* stream) {
    if (!q || !K || !V || !out) return MKV_ERR_INVALID_ARG;
    if (batch < 1 || q_heads < 1 || kv_heads < 1 || q_heads % kv_heads) return MKV_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return MKV_ERR_UNSUPPORTED;
    if (kv_dtype != MKV_BF16 && kv_dtype != MKV_F32) return MKV_ERR_INVALID_ARG;
    if (out_dtype != MKV_BF16 && out_dtype != MKV_F32) return MKV_ERR_INVALID_ARG;
    if (n_tokens < 1 || kv_rows < n_tokens) return MKV_ERR_INVALID_ARG;
    if (device < 0 || device >= kNaMaxDevices) return MKV_ERR_INVALID_ARG;
    const int G = q_heads / kv_heads;
    if (G > 8) return MKV_ERR_UNSUPPORTED;
    // the static scratch bounds the problem: refuse what does not fit
    const long long splits = ((long long)n_tokens + kNaChunkRows - 1) / kNaChunkRows;
    const long long units = (long long)batch * kv_heads;
    if (splits > 64 || units > kNaMaxUnits || (long long)batch * q_heads * splits > kNaMaxPartRows)
        return MKV_ERR_CAPACITY;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return MKV_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return MKV_ERR_CUDA;
    mkv_status rc = MKV_OK;
    if (!g_na_ptr[device]) {
        // once per device, with that device current: the array's name is only a host-side
        // handle, the kernel needs the address the runtime reports for this device
        float* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_na_scratch) != cudaSuccess || !ptr) rc = MKV_ERR_CUDA;
        else g_na_ptr[device] = ptr;
    }
    if (rc == MKV_OK) {
        NaParams p;
        p.q = q; p.K = K; p.V = V; p.out = out;
        p.parts = g_na_ptr[device];
        p.tickets = reinterpret_cast<int*>(g_na_ptr[device] + (size_t)kNaMaxPartRows * kNaPartStride);
        p.batch = batch; p.q_heads = q_heads; p.kv_heads = kv_heads; p.group = G;
        p.n_tokens = n_tokens; p.kv_rows = kv_rows; p.splits = (int)splits;
        p.scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
        p.out_f32 = (out_dtype == MKV_F32);
        cudaStream_t st = (cudaStream_t)stream;
        // tickets must start at zero whatever an earlier call left there
        if (cudaMemsetAsync(p.tickets, 0, sizeof(int) * (size_t)units, st) != cudaSuccess) rc = MKV_ERR_CUDA;
        if (rc == MKV_OK) {
            const dim3 grid((unsigned)splits, (unsigned)units), block(kNaThreads);
            if (kv_dtype == MKV_BF16) {
                if (head_dim == 128) na_attend_kernel<__nv_bfloat16, 128><<<grid, block, 0, st>>>(p);
                else na_attend_kernel<__nv_bfloat16, 64><<<grid, block, 0, st>>>(p);
            } else {
                if (head_dim == 128) na_attend_kernel<float, 128><<<grid, block, 0, st>>>(p);
                else na_attend_kernel<float, 64><<<grid, block, 0, st>>>(p);
            }
            if (cudaGetLastError() != cudaSuccess) rc = MKV_ERR_CUDA;
        }
    }
    if (prev >= 0 && prev != device) cudaSetDevice(prev);
    return rc;
}
