// Scoring exactly as Eq. 4 prints it: the attention a decode token receives is averaged over
// ALL H query heads of the layer, the layer keeps ONE importance vector per sequence, and all
// KV heads evict the same tokens (score mode MKV_SCORE_LAYER_MEAN with more than one KV
// head).  The streaming kernels run unchanged but leave the unit tails out; this kernel then
// does for all KV heads of a sequence what a unit tail does for one.  One CTA per
// (sequence, KV head) handles that head's share; the CTA that finishes last for a sequence
// (a ticket) does the part that needs all heads:
//   per KV head: the fresh token's logits, the cross-split combine, `out`          (Eq. 2)
//                and, per decode token, the sum over its G heads of 2^(s - M_h) / L_h
//   per decode token: abar = (1/H) sum of those sums over the KV heads               (Eq. 4)
//   I <- beta * I + abar, the fresh token starting from 0                            (Eq. 5, 6)
//   one selection of the overflow-many lowest (score bits, position id) keys         (Eq. 7, 8)
//   the same append / hole filling in every KV head's pool                           (Eq. 9)
// Every KV head's unit holds an equal copy of the scores, position ids and counts, so the
// streaming kernels and the inspection calls need not know about the mode.
#include "mkv_launch.h"
#include "mkv_tail.cuh"

namespace mkv {
namespace {

constexpr int kLtThreads = 256;
constexpr int kLtWarps = kLtThreads / 32;
constexpr int kLtMaxHeads = 128;     // query heads of a layer this kernel is built for

template <typename T>
__global__ void __launch_bounds__(kLtThreads) layer_tail_kernel(const Params p) {
    __shared__ float sM[kLtMaxHeads], sInvL[kLtMaxHeads], sSnew[kLtMaxHeads], sWnew[kLtMaxHeads];
    __shared__ float sW[kMaxParts][kMaxGroup], sPl[kMaxParts][kMaxGroup];
    __shared__ unsigned long long red_key[kLtWarps];
    __shared__ int red_slot[kLtWarps];
    __shared__ int hist[256];
    __shared__ int cnt[3][kLtWarps];
    __shared__ int misc[4];

    const LayerDev& L = p.L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = p.group, D = p.head_dim, cap = p.cap, ls = p.lstride, Hkv = p.kv_heads, Hq = p.q_heads;
    const int rowb = D * (int)sizeof(T);
    const int b = blockIdx.x / Hkv, u0 = b * Hkv;
    const int n_old = min(L.n_dec[u0], cap - 1);
    const int n = n_old + 1;
    const int t = L.unit_step[u0];
    const int k = max(0, n - p.budget);
    __shared__ int s_last;
    // the streaming kernel of this step has finished and has counted itself: its parity is
    // that of the launch before the count now stored
    const int par = (int)((__ldcg(&L.launch_no[0]) & 1u) ^ 1u);

    // ---- this CTA's KV head: fresh logits, combine, out, and its heads' share of Eq. 4 ------------
    {
        const int g = blockIdx.x - b * Hkv;
        const int u = u0 + g;
        const int P = min(__ldcg(&L.cnt[(size_t)par * L.n_units + u].y), kMaxParts), part0 = u * kMaxParts;
        const T* qrow = reinterpret_cast<const T*>(p.q) + ((size_t)b * Hq + (size_t)g * G) * D;
        const T* knew = reinterpret_cast<const T*>(p.k_new) + (size_t)u * D;
        const T* vnew = reinterpret_cast<const T*>(p.v_new) + (size_t)u * D;
        for (int h = warp; h < G; h += kLtWarps) {
            float a = 0.f;
            for (int e = lane; e < D; e += 32) a = fmaf(to_f32(qrow[(size_t)h * D + e]), to_f32(knew[e]), a);
#pragma unroll
            for (int off = 16; off; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            if (lane == 0) sSnew[g * G + h] = a * p.scale_log2;
        }
        for (int e = tid; e < P * kMaxGroup; e += kLtThreads) {
            const int q = e / kMaxGroup, h = e - q * kMaxGroup;
            if (h < G) {
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(&L.part_ml[((size_t)(part0 + q) * G + h) * 2]));
                sW[q][h] = ml.x;
                sPl[q][h] = ml.y;
            }
        }
        __syncthreads();
        if (tid < G) {
            const int hq = g * G + tid;
            float M = sSnew[hq];
            for (int q = 0; q < P; ++q) M = fmaxf(M, sW[q][tid]);
            float Lsum = 0.f;
            for (int q = 0; q < P; ++q) {
                const float w = fast_exp2(sW[q][tid] - M);
                sW[q][tid] = w;
                Lsum = fmaf(sPl[q][tid], w, Lsum);
            }
            const float wn = fast_exp2(sSnew[hq] - M);
            Lsum += wn;
            sWnew[hq] = wn;
            sM[hq] = M;
            sInvL[hq] = Lsum > 0.f ? 1.0f / Lsum : 0.f;
        }
        __syncthreads();
        const size_t obase = ((size_t)b * Hq + (size_t)g * G) * D;
        for (int idx = tid; idx < G * D; idx += kLtThreads) {
            const int h = idx / D;
            float acc = to_f32(vnew[idx - h * D]) * sWnew[g * G + h];
            for (int q = 0; q < P; ++q)
                acc = fmaf(__ldcg(&L.part_o[(size_t)(part0 + q) * G * D + idx]), sW[q][h], acc);
            acc *= sInvL[g * G + h];
            if (p.out_f32) reinterpret_cast<float*>(p.out)[obase + idx] = acc;
            else reinterpret_cast<__nv_bfloat16*>(p.out)[obase + idx] = __float2bfloat16_rn(acc);
        }
        // sum over this KV head's G query heads of the normalised probabilities, per decode token
        // (the fresh token last), parked in the unit's row of the compaction scratch
        float* part = reinterpret_cast<float*>(L.list_b + (size_t)u * cap);
        const float* lgu = L.logit + ((size_t)b * Hq + (size_t)g * G) * ls;
        for (int i = tid; i < n_old; i += kLtThreads) {
            float s = 0.f;
            for (int h = 0; h < G; ++h) s = fmaf(fast_exp2(__ldcg(&lgu[(size_t)h * ls + i]) - sM[g * G + h]), sInvL[g * G + h], s);
            part[i] = s;
        }
        if (tid == 0) {
            float s = 0.f;
            for (int h = 0; h < G; ++h) s = fmaf(sWnew[g * G + h], sInvL[g * G + h], s);
            part[n_old] = s;
        }
        __threadfence();
        __syncthreads();
    }
    // The CTA that finishes last for the sequence goes on (and leaves the ticket at zero).
    if (tid == 0) {
        s_last = (atomicAdd(&L.seq_ticket[b], 1) == Hkv - 1);
        if (s_last) L.seq_ticket[b] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- all heads: head mean, momentum update -----------------------------------------------
    const float inv_h = 1.0f / (float)Hq;
    float ab_new = 0.f;
    for (int g = 0; g < Hkv; ++g) ab_new += __ldcg(reinterpret_cast<const float*>(L.list_b + (size_t)(u0 + g) * cap) + n_old);
    ab_new *= inv_h;                                   // Eq. 6: I_fresh = alpha * 0 + abar_fresh
    const unsigned long long key_new = ((unsigned long long)__float_as_uint(ab_new) << 32) | (unsigned)t;
    unsigned long long* keys = L.keys + (size_t)u0 * cap;
    const float* score0 = L.score + (size_t)u0 * ls;
    const int32_t* pos0 = L.pos + (size_t)u0 * ls;
    unsigned long long best_key = ~0ull;
    int best_slot = -1;
    for (int i = tid; i < n_old; i += kLtThreads) {
        float s = 0.f;
        for (int g = 0; g < Hkv; ++g) s += __ldcg(reinterpret_cast<const float*>(L.list_b + (size_t)(u0 + g) * cap) + i);
        const float ab = s * inv_h;
        const float nw = fmaf(p.beta, score0[i], ab);
        for (int g = 0; g < Hkv; ++g) {
            L.score[(size_t)(u0 + g) * ls + i] = nw;
            if (L.abar) L.abar[(size_t)(u0 + g) * cap + i] = ab;
        }
        const unsigned long long key = ((unsigned long long)__float_as_uint(nw) << 32) | (unsigned)pos0[i];
        if (k > 1) keys[i] = key;
        if (key < best_key) { best_key = key; best_slot = i; }
    }
    if (tid == kLtThreads - 1) {                       // the fresh token sits (virtually) in slot n_old
        if (key_new < best_key) { best_key = key_new; best_slot = n_old; }
        if (L.abar)
            for (int g = 0; g < Hkv; ++g) L.abar[(size_t)(u0 + g) * cap + n_old] = ab_new;
    }
    if (tid < Hkv) {
        const int u = u0 + tid;
        L.n_prev[u] = n; L.ev_k[u] = k; L.n_dec[u] = n - k; L.unit_step[u] = t + 1;
        rewind_unit(L, u, par);
    }

    // the fresh row of KV head g into slot `dst` of its pool, with the shared score and id
    auto place_fresh = [&](int dst) {
        for (int g = warp; g < 2 * Hkv; g += kLtWarps) {
            const int u = u0 + (g >> 1);
            const size_t ubase = (size_t)u * cap * rowb;
            if (g & 1) store_row_swizzled(L.Vd, ubase, rowb, reinterpret_cast<const T*>(p.v_new) + (size_t)u * D, dst, lane);
            else store_row_swizzled(L.Kd, ubase, rowb, reinterpret_cast<const T*>(p.k_new) + (size_t)u * D, dst, lane);
        }
        if (tid < Hkv) { L.score[(size_t)(u0 + tid) * ls + dst] = ab_new; L.pos[(size_t)(u0 + tid) * ls + dst] = t; }
    };

    if (k != 1) {
        place_fresh(n_old);                            // append at the end
        if (tid == 0) keys[n_old] = key_new;
        if (k == 0) return;
    }
    if (k == 1) {
        for (int off = 16; off; off >>= 1) {
            const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best_key, off);
            const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
            if (ok < best_key) { best_key = ok; best_slot = os; }
        }
        if (lane == 0) { red_key[warp] = best_key; red_slot[warp] = best_slot; }
        __syncthreads();     // also orders every score write before the stores below
        unsigned long long kk = red_key[0];
        int e = red_slot[0];
        for (int w2 = 1; w2 < kLtWarps; ++w2)
            if (red_key[w2] < kk) { kk = red_key[w2]; e = red_slot[w2]; }
        if (tid < Hkv) {
            L.ev_pos[(size_t)(u0 + tid) * cap] = (int32_t)(unsigned)(kk & 0xffffffffu);
            L.ev_score[(size_t)(u0 + tid) * cap] = __uint_as_float((unsigned)(kk >> 32));
        }
        if (e != n_old) place_fresh(e);                // the fresh row lands in the hole
        return;
    }

    // ---- overflow > 1: radix select of the k-th smallest key, then ordered hole filling ---------
    __syncthreads();
    unsigned long long prefix = 0ull, mask = 0ull;
    int want = k - 1;
    for (int pass = 7; pass >= 0; --pass) {
        for (int i = tid; i < 256; i += kLtThreads) hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += kLtThreads) {
            const unsigned long long key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&hist[(int)((key >> (8 * pass)) & 255ull)], 1);
        }
        __syncthreads();
        if (tid == 0) {
            int cum = 0, sel = 255;
            for (int bin = 0; bin < 256; ++bin) {
                const int c = hist[bin];
                if (want < cum + c) { sel = bin; break; }
                cum += c;
            }
            misc[0] = sel;
            misc[1] = want - cum;
        }
        __syncthreads();
        prefix |= (unsigned long long)misc[0] << (8 * pass);
        mask |= 255ull << (8 * pass);
        want = misc[1];
    }
    const unsigned long long kth = prefix;
    const int n_new = n - k;
    int32_t* holes = L.list_a + (size_t)u0 * cap;
    int32_t* movers = L.list_b + (size_t)u0 * cap;
    int hc = 0, mc = 0, ec = 0;
    for (int base = 0; base < n; base += kLtThreads) {
        const int i = base + tid;
        const bool valid = i < n;
        const unsigned long long key = valid ? keys[i] : ~0ull;
        const bool ev = valid && key <= kth;
        const bool hole = ev && i < n_new;
        const bool mover = valid && !ev && i >= n_new;
        const unsigned bh = __ballot_sync(0xffffffffu, hole);
        const unsigned bm = __ballot_sync(0xffffffffu, mover);
        const unsigned be = __ballot_sync(0xffffffffu, ev);
        const unsigned lt = (1u << lane) - 1u;
        if (lane == 0) { cnt[0][warp] = __popc(bh); cnt[1][warp] = __popc(bm); cnt[2][warp] = __popc(be); }
        __syncthreads();
        int ph = 0, pm = 0, pe = 0, th = 0, tm = 0, te = 0;
        for (int w2 = 0; w2 < kLtWarps; ++w2) {
            if (w2 < warp) { ph += cnt[0][w2]; pm += cnt[1][w2]; pe += cnt[2][w2]; }
            th += cnt[0][w2]; tm += cnt[1][w2]; te += cnt[2][w2];
        }
        if (hole) holes[hc + ph + __popc(bh & lt)] = i;
        if (mover) movers[mc + pm + __popc(bm & lt)] = i;
        if (ev) {
            const int j = ec + pe + __popc(be & lt);
            for (int g = 0; g < Hkv; ++g) {
                L.ev_pos[(size_t)(u0 + g) * cap + j] = (int32_t)(unsigned)(key & 0xffffffffu);
                L.ev_score[(size_t)(u0 + g) * cap + j] = __uint_as_float((unsigned)(key >> 32));
            }
        }
        hc += th; mc += tm; ec += te;
        __syncthreads();
    }
    if (hc != mc || ec != k) {
        if (tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
        return;
    }
    for (int j = warp; j < hc * Hkv; j += kLtWarps) {
        const int g = j / hc, m = j - g * hc;
        const int src = movers[m], dst = holes[m];
        const int u = u0 + g;
        const size_t ubase = (size_t)u * cap * rowb;
        copy_row_swizzled(L.Kd, ubase, rowb, src, dst, lane);
        copy_row_swizzled(L.Vd, ubase, rowb, src, dst, lane);
        if (lane == 0) {
            L.score[(size_t)u * ls + dst] = L.score[(size_t)u * ls + src];
            L.pos[(size_t)u * ls + dst] = L.pos[(size_t)u * ls + src];
        }
    }
}

}  // namespace

bool layer_tail_supported(int q_heads, int group) { return q_heads <= kLtMaxHeads && group <= kMaxGroup; }

cudaError_t launch_layer_tail(const Params& p, int kv_dtype, cudaStream_t st) {
    const unsigned grid = (unsigned)(p.batch * p.kv_heads);
    if (kv_dtype == 0) layer_tail_kernel<__nv_bfloat16><<<grid, kLtThreads, 0, st>>>(p);
    else layer_tail_kernel<float><<<grid, kLtThreads, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mkv
