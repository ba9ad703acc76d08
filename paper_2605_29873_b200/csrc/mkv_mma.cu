// Tensor-core split-KV decode attention for bf16 caches, head_dim 128, G <= 8: the hot
// path of the Llama-3.1-8B- and Qwen2.5-7B-shaped workloads.
//
// Decode attention at GQA group 4-7 is bound by streaming K and V from HBM once per KV
// head; the kernel is built around that stream.
//   * Persistent CTAs (two per SM) pull items from an atomic work counter, so the grid is
//     a multiple of the SM count and load balance does not depend on sequence lengths.
//   * One producer thread per CTA issues bulk asynchronous copies (the non-tensor TMA
//     form, no multicast) of 64-row K and V tiles, 16 KB each, into a ring of shared
//     memory stages; completion is signalled on an mbarrier (complete_tx).  The cache
//     rows are already chunk-permuted in HBM, so a straight copy lands a layout that
//     ldmatrix reads without bank conflicts.  The producer keeps prefetching across item
//     boundaries and while the consumers run a unit's tail.
//   * Four consumer warps each own 16 rows of a tile.  S = Q K^T and O += P V use
//     mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the G query heads padded to the
//     16-row M dimension: this is not a GEMM reshaping for the sake of tensor cores, it
//     takes the per-row instruction count from ~60 (scalar FMA + shuffles) to ~7 so that
//     issue slots never limit the HBM stream, for G = 7 as well as G = 4.  The softmax
//     runs in registers in fp32 (quad shuffles for the row maximum); P enters the second
//     mma as hi + lo bf16 halves, so the rounding of P to bf16 does not reach `out`.
//   * Raw fp32 logits of decode-pool tokens are stored (4 bytes per head and token) for
//     the tail, which needs the global log-sum-exp before it can normalise them (Eq. 4).
//   * At the end of an item the four warps merge (m, l, O) through shared memory, write
//     one partial and take the unit's ticket; the last ticket holder runs the tail.
// Every wait is bounded: on expiry the kernel records MKV_ERR_TIMEOUT and drains.
#include "mkv_launch.h"
#include "mkv_ptx.cuh"
#include "mkv_tail.cuh"

namespace mkv {
namespace {

constexpr int kTileRows = 64;
constexpr int kRowB = 256;                                // 128 bf16
constexpr int kTileBytes = kTileRows * kRowB;             // 16 KB (K or V)
constexpr int kStageBytes = 2 * kTileBytes;               // K then V
constexpr int kConsumerWarps = 4;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;
constexpr int kMaxStages = 8;
constexpr unsigned long long kWaitNs = 4000000000ull;     // 4 s

struct StageMeta {
    int item;       // -1: no more work
    int unit;
    int seg;
    int row;        // slot of the tile's first row inside its pool (multiple of 16)
    int cnt_pool;   // rows copied from the pool
    int fresh_row;  // tile row that takes the step's fresh token, or -1
    int first, last;
};

template <int GR>
struct MergeSmem {
    static constexpr int NH = GR / 4;          // column halves merged one after the other
    static constexpr int HC = 128 / NH;
    float xm[kConsumerWarps][GR];
    float xl[kConsumerWarps][GR];
    float xo[kConsumerWarps][GR][HC + 4];
};

template <int GR>
union alignas(16) ScratchSmem {
    TailSmem<kConsumers> tail;
    MergeSmem<GR> merge;
};

struct Control {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    StageMeta meta[kMaxStages];
    int abort_flag;
    int last_flag;
};

template <int GR>
constexpr size_t smem_bytes(int nst) {
    return (size_t)nst * kStageBytes + sizeof(ScratchSmem<GR>) + sizeof(Control);
}

__device__ inline void note_timeout(const Params& p, Control* ctl) {
    atomicCAS(p.status, kStatusOk, kStatusTimeout);
    *reinterpret_cast<volatile int*>(&ctl->abort_flag) = 1;
}

template <int GR>
__global__ void __launch_bounds__(kThreads, 2) mma_kernel(const Params p, const int nst) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* const stages = smem;
    ScratchSmem<GR>* const scratch = reinterpret_cast<ScratchSmem<GR>*>(smem + (size_t)nst * kStageBytes);
    Control* const ctl = reinterpret_cast<Control*>(smem + (size_t)nst * kStageBytes + sizeof(ScratchSmem<GR>));

    const LayerDev& L = p.L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool dec = (p.mode == kModeDecode);
    const int G = p.group;

    if (tid == 0) {
        for (int s = 0; s < nst; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), kConsumerWarps);
        }
        ctl->abort_flag = 0;
        ctl->last_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ================================ producer =====================================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            while (ok) {
                const int it = atomicAdd(&L.sched[0], 1);
                if (it >= L.n_items) break;
                const int4 v = __ldg(reinterpret_cast<const int4*>(&L.items[it]));
                const int u = v.x, row0 = v.y, rows = v.z, seg = v.w;
                int pool_rows, fresh = -1;
                const uint8_t *kb, *vb;
                if (seg == 0) {
                    pool_rows = rows;
                    kb = L.Kp + ((size_t)u * p.max_prefill + row0) * kRowB;
                    vb = L.Vp + ((size_t)u * p.max_prefill + row0) * kRowB;
                } else {
                    const int n_old = min(L.n_dec[u], p.cap - (dec ? 1 : 0));
                    pool_rows = max(0, min(rows, n_old - row0));
                    if (dec && n_old >= row0 && n_old < row0 + rows) fresh = n_old - row0;
                    kb = L.Kd + ((size_t)u * p.cap + row0) * kRowB;
                    vb = L.Vd + ((size_t)u * p.cap + row0) * kRowB;
                }
                const int total = pool_rows + (fresh >= 0 ? 1 : 0);
                const int ntiles = max(1, (total + kTileRows - 1) / kTileRows);
                for (int t = 0; t < ntiles; ++t) {
                    const uint32_t fb = ptx::smem_u32(&ctl->full[stage]);
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, kWaitNs)) {
                        note_timeout(p, ctl);
                        ok = false;
                        break;
                    }
                    if (*reinterpret_cast<volatile int*>(&ctl->abort_flag)) { ok = false; break; }
                    const int r = t * kTileRows;
                    const int cnt = max(0, min(kTileRows, pool_rows - r));
                    StageMeta& mt = ctl->meta[stage];
                    mt.item = it; mt.unit = u; mt.seg = seg; mt.row = row0 + r; mt.cnt_pool = cnt;
                    mt.fresh_row = (fresh >= r && fresh < r + kTileRows) ? fresh - r : -1;
                    mt.first = (t == 0); mt.last = (t == ntiles - 1);
                    if (cnt > 0) {
                        const uint32_t dstK = ptx::smem_u32(stages + (size_t)stage * kStageBytes);
                        ptx::mbar_arrive_expect_tx(fb, (uint32_t)cnt * 2u * kRowB);
                        ptx::bulk_g2s(dstK, kb + (size_t)r * kRowB, (uint32_t)cnt * kRowB, fb);
                        ptx::bulk_g2s(dstK + kTileBytes, vb + (size_t)r * kRowB, (uint32_t)cnt * kRowB, fb);
                    } else {
                        ptx::mbar_arrive(fb);
                    }
                    if (++stage == nst) { stage = 0; phase ^= 1u; }
                }
            }
            if (ok) {
                if (ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, kWaitNs)) {
                    ctl->meta[stage].item = -1;
                    ptx::mbar_arrive(ptx::smem_u32(&ctl->full[stage]));
                } else {
                    note_timeout(p, ctl);
                }
            }
        }
        __syncwarp();
    } else {
        // ================================ consumers ====================================
        int stage = 0;
        uint32_t phase = 0;
        float oacc[16][4];
        float m_run = kNegBig, l_run = 0.f;
        uint32_t qa[8][2];
        const int head = lane >> 2, tk0 = 2 * (lane & 3);
        const int mi = lane >> 3, rr = lane & 7;
        const int blk0 = warp * 16;
#pragma unroll
        for (int j = 0; j < 16; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) { qa[ks][0] = qa[ks][1] = 0u; }

        for (;;) {
            if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->full[stage]), phase, kWaitNs)) {
                if (lane == 0) note_timeout(p, ctl);
                break;
            }
            const StageMeta mt = ctl->meta[stage];
            if (mt.item < 0) break;
            const int u = mt.unit;
            const int b = u / p.kv_heads, g = u - b * p.kv_heads;
            if (mt.first) {
                const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(p.q) +
                                            ((size_t)b * p.q_heads + (size_t)g * G + min(head, G - 1)) * 128 + tk0;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t x0 = __ldg(reinterpret_cast<const uint32_t*>(qrow + 16 * ks));
                    const uint32_t x1 = __ldg(reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8));
                    qa[ks][0] = head < G ? x0 : 0u;
                    qa[ks][1] = head < G ? x1 : 0u;
                }
                m_run = kNegBig; l_run = 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }
            }
            uint8_t* const sK = stages + (size_t)stage * kStageBytes;
            uint8_t* const sV = sK + kTileBytes;
            const int nv = mt.cnt_pool + (mt.fresh_row >= 0 ? 1 : 0);
            bool wrote = false;
            if (mt.fresh_row >= 0 && (mt.fresh_row >> 4) == warp) {
                // Algorithm 1 append: the fresh token joins the tile from k_new / v_new and is
                // stored into its pool slot for the following steps.
                const int c = lane & 15;
                const bool isv = lane >= 16;
                const uint4 val = *reinterpret_cast<const uint4*>(
                    reinterpret_cast<const uint8_t*>(isv ? p.v_new : p.k_new) + (size_t)u * kRowB + c * 16);
                const int fr = mt.fresh_row;
                const uint32_t off = (uint32_t)fr * kRowB + (uint32_t)((c ^ (fr & 7)) << 4);
                *reinterpret_cast<uint4*>((isv ? sV : sK) + off) = val;
                const int slot = mt.row + fr;
                *reinterpret_cast<uint4*>((isv ? L.Vd : L.Kd) + ((size_t)u * p.cap + slot) * kRowB +
                                          (uint32_t)((c ^ (slot & 7)) << 4)) = val;
                wrote = true;
            }
            if (nv > blk0 && nv < blk0 + 16) {
                // rows past the valid ones enter the second mma with probability 0: their V
                // bytes must be finite, so clear them (stale shared memory may hold anything)
                const int nz = (blk0 + 16 - nv) * 16;
                for (int idx = lane; idx < nz; idx += 32)
                    *reinterpret_cast<uint4*>(sV + (size_t)(nv + (idx >> 4)) * kRowB + ((idx & 15) << 4)) =
                        make_uint4(0u, 0u, 0u, 0u);
                wrote = true;
            }
            __syncwarp();

            if (nv > blk0) {
                // ---------------- S = Q K^T for 16 heads (padded) x 16 tokens ----------------
                float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                const uint32_t kbase = ptx::smem_u32(sK) + (uint32_t)(blk0 + (mi >> 1) * 8 + rr) * kRowB;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    uint32_t b00, b01, b10, b11;
                    ptx::ldmatrix_x4(kbase + (uint32_t)(((2 * ks + (mi & 1)) ^ rr) << 4), b00, b01, b10, b11);
                    ptx::mma_bf16(sacc[0], qa[ks][0], 0u, qa[ks][1], 0u, b00, b01);
                    ptx::mma_bf16(sacc[1], qa[ks][0], 0u, qa[ks][1], 0u, b10, b11);
                }
                // ---------------- online softmax in registers (fp32) -------------------------
                float s[4] = {sacc[0][0], sacc[0][1], sacc[1][0], sacc[1][1]};
                const int trow[4] = {blk0 + tk0, blk0 + tk0 + 1, blk0 + tk0 + 8, blk0 + tk0 + 9};
#pragma unroll
                for (int i = 0; i < 4; ++i) s[i] = (trow[i] < nv) ? s[i] * p.scale_log2 : kNegBig;
                if (dec && mt.seg == 1 && head < G) {
                    float* lg = L.logit + ((size_t)b * p.q_heads + (size_t)g * G + head) * p.cap + mt.row;
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (trow[i] < nv) lg[trow[i]] = s[i];
                }
                float mx = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float sc = fast_exp2(m_run - m_new);
                float pr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) pr[i] = fast_exp2(s[i] - m_new);
                l_run = fmaf(l_run, sc, (pr[0] + pr[1]) + (pr[2] + pr[3]));
                m_run = m_new;
                if (sc != 1.0f) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) { oacc[j][0] *= sc; oacc[j][1] *= sc; }
                }
                // P = hi + lo in bf16: the product with V then carries ~16 mantissa bits of P
                const uint32_t ahi0 = ptx::pack_bf16x2(pr[0], pr[1]);
                const uint32_t ahi2 = ptx::pack_bf16x2(pr[2], pr[3]);
                const uint32_t alo0 = ptx::pack_bf16x2(pr[0] - __uint_as_float(ahi0 << 16),
                                                       pr[1] - __uint_as_float(ahi0 & 0xffff0000u));
                const uint32_t alo2 = ptx::pack_bf16x2(pr[2] - __uint_as_float(ahi2 << 16),
                                                       pr[3] - __uint_as_float(ahi2 & 0xffff0000u));
                // ---------------- O += P V ------------------------------------------------------
                const uint32_t vbase = ptx::smem_u32(sV) + (uint32_t)(blk0 + (mi & 1) * 8 + rr) * kRowB;
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    uint32_t b0, b1, b2, b3;
                    ptx::ldmatrix_x4_trans(vbase + (uint32_t)(((j + (mi >> 1)) ^ rr) << 4), b0, b1, b2, b3);
                    ptx::mma_bf16(oacc[j], ahi0, 0u, ahi2, 0u, b0, b1);
                    ptx::mma_bf16(oacc[j], alo0, 0u, alo2, 0u, b0, b1);
                    ptx::mma_bf16(oacc[j + 1], ahi0, 0u, ahi2, 0u, b2, b3);
                    ptx::mma_bf16(oacc[j + 1], alo0, 0u, alo2, 0u, b2, b3);
                }
            }
            if (wrote) ptx::fence_proxy_async();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->empty[stage]));
            if (++stage == nst) { stage = 0; phase ^= 1u; }

            if (mt.last) {
                // ---------------- item end: merge the four warps, one partial, ticket -----------
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
                MergeSmem<GR>& mg = scratch->merge;
                constexpr int NH = MergeSmem<GR>::NH, HC = MergeSmem<GR>::HC;
                if ((lane & 3) == 0 && head < GR) { mg.xm[warp][head] = m_run; mg.xl[warp][head] = l_run; }
                const size_t part = (size_t)mt.item;
#pragma unroll
                for (int half = 0; half < NH; ++half) {
                    if (head < GR) {
#pragma unroll
                        for (int jj = 0; jj < 16 / NH; ++jj) {
                            const int j = half * (16 / NH) + jj;
                            *reinterpret_cast<float2*>(&mg.xo[warp][head][jj * 8 + tk0]) =
                                make_float2(oacc[j][0], oacc[j][1]);
                        }
                    }
                    bar_sync(1, kConsumers);
                    for (int idx = tid; idx < G * HC; idx += kConsumers) {
                        const int row = idx / HC, col = idx - row * HC;
                        float M = mg.xm[0][row];
#pragma unroll
                        for (int w = 1; w < kConsumerWarps; ++w) M = fmaxf(M, mg.xm[w][row]);
                        float acc = 0.f, ls = 0.f;
#pragma unroll
                        for (int w = 0; w < kConsumerWarps; ++w) {
                            const float wsc = fast_exp2(mg.xm[w][row] - M);
                            acc = fmaf(mg.xo[w][row][col], wsc, acc);
                            ls = fmaf(mg.xl[w][row], wsc, ls);
                        }
                        L.part_o[(part * G + row) * 128 + half * HC + col] = acc;
                        if (half == 0 && col == 0) {
                            L.part_ml[(part * G + row) * 2] = M;
                            L.part_ml[(part * G + row) * 2 + 1] = ls;
                        }
                    }
                    __threadfence();
                    bar_sync(1, kConsumers);
                }
                if (tid == 0) ctl->last_flag = (atomicAdd(&L.ticket[u], 1) == L.unit_nparts[u] - 1);
                bar_sync(1, kConsumers);
                if (ctl->last_flag) {
                    __threadfence();
                    unit_tail<kConsumers, 1>(p, u, scratch->tail, tid, kRowB);
                    bar_sync(1, kConsumers);
                }
            }
        }
    }
    __syncthreads();
    if (tid == 0) grid_epilogue(p, gridDim.x);
}

int g_stages = 3;

}  // namespace

bool mma_supported(int kv_dtype, int head_dim, int group) {
    return kv_dtype == 0 && head_dim == 128 && group >= 1 && group <= 8;
}

cudaError_t mma_configure() {
    if (const char* e = std::getenv("MKV_STAGES")) g_stages = max(2, min(kMaxStages, atoi(e)));
    cudaError_t err = cudaFuncSetAttribute(mma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem_bytes<4>(g_stages));
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(mma_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)smem_bytes<8>(g_stages));
}

cudaError_t launch_mma(const Params& p, int n_ctas, cudaStream_t st) {
    if (p.L.n_items <= 0) return cudaSuccess;
    if (p.group <= 4) mma_kernel<4><<<n_ctas, kThreads, smem_bytes<4>(g_stages), st>>>(p, g_stages);
    else mma_kernel<8><<<n_ctas, kThreads, smem_bytes<8>(g_stages), st>>>(p, g_stages);
    return cudaGetLastError();
}

}  // namespace mkv
