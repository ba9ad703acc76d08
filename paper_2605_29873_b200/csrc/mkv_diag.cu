// Recency-window attention diagnostics (Sec. 3.2 and Sec. 7.1 of the paper: how the attention
// of a step is spread over the most recently decoded tokens).  Not part of the decode step:
// a kernel of its own over the head-averaged probabilities (Eq. 4) and position ids that a step
// records when the context was created with MKV_FLAG_RECORD_PROBS, run on demand.
//
// One CTA per (sequence, KV head) unit.  The tokens of the window -- position id among the last
// W step ids, the step's own token included -- are collected in shared memory, sorted by
// attention (bitonic network, descending), and summed up in that order in fp64:
//   mass  = attention the window received, a share of 1
//   curve[j] = share of `mass` held by the j+1 most attended tokens of the window
#include "mkv_launch.h"

namespace mkv {
namespace {

constexpr int kDiagThreads = 256;

__global__ void __launch_bounds__(kDiagThreads) diag_kernel(const LayerDev L, const int cap, const int window,
                                                            const int npow2, float* __restrict__ mass,
                                                            int32_t* __restrict__ count, float* __restrict__ curve) {
    extern __shared__ float vals[];                    // [npow2]
    __shared__ int s_cnt;
    __shared__ double s_part[kDiagThreads];
    const int u = blockIdx.x, tid = threadIdx.x;
    const int steps = L.unit_step[u];                  // steps completed: the last one had id steps - 1
    const int n = steps > 0 ? min(L.n_prev[u], cap) : 0;
    const int t = steps - 1;
    if (tid == 0) s_cnt = 0;
    for (int i = tid; i < npow2; i += kDiagThreads) vals[i] = -1.0f;   // below every probability
    __syncthreads();
    const float* ab = L.abar + (size_t)u * cap;
    const int32_t* ps = L.abar_pos + (size_t)u * cap;
    for (int i = tid; i < n; i += kDiagThreads) {
        const int age = t - ps[i];
        if (age >= 0 && age < window) {
            const int j = atomicAdd(&s_cnt, 1);
            if (j < npow2) vals[j] = ab[i];
        }
    }
    __syncthreads();
    const int cnt = min(s_cnt, npow2);
    // bitonic sort, descending (the fill value sinks to the end)
    for (int k = 2; k <= npow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < npow2; i += kDiagThreads) {
                const int x = i ^ j;
                if (x > i) {
                    const float a = vals[i], b = vals[x];
                    const bool desc = (i & k) == 0;
                    if (desc ? (a < b) : (a > b)) { vals[i] = b; vals[x] = a; }
                }
            }
            __syncthreads();
        }
    }
    // running sums in sorted order: every thread a contiguous piece, then the pieces' offsets
    const int per = (npow2 + kDiagThreads - 1) / kDiagThreads;
    const int lo = min(tid * per, cnt), hi = min(lo + per, cnt);
    double local = 0.0;
    for (int i = lo; i < hi; ++i) local += (double)vals[i];
    s_part[tid] = local;
    __syncthreads();
    double before = 0.0, total = 0.0;
    for (int w = 0; w < kDiagThreads; ++w) {
        if (w < tid) before += s_part[w];
        total += s_part[w];
    }
    double run = before;
    float* row = curve + (size_t)u * window;
    for (int i = lo; i < hi; ++i) {
        run += (double)vals[i];
        row[i] = total > 0.0 ? (float)(run / total) : 0.f;
    }
    for (int i = cnt + tid; i < window; i += kDiagThreads) row[i] = 0.f;   // beyond the window's tokens
    if (tid == 0) { mass[u] = (float)total; count[u] = cnt; }
}

}  // namespace

// Largest window-or-capacity the sort holds in shared memory without opting in to more.
int diag_max_tokens() { return 8192; }

cudaError_t launch_diag(const LayerDev& L, int cap, int window, float* mass, int32_t* count, float* curve,
                        cudaStream_t st) {
    const int need = window < cap ? window : cap;
    int npow2 = 2;
    while (npow2 < need) npow2 <<= 1;
    diag_kernel<<<(unsigned)L.n_units, kDiagThreads, (size_t)npow2 * sizeof(float), st>>>(L, cap, window, npow2, mass,
                                                                                         count, curve);
    return cudaGetLastError();
}

}  // namespace mkv
