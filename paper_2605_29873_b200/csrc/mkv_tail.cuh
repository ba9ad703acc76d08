// Tail of one unit (sequence b, KV head g), run by the thread group that delivered the
// unit's last partial.  In order:
//   0. the fresh token of the step (Algorithm 1, append): its logit q_h . k_new / sqrt(d)
//      for the G heads; it takes part in the softmax as one more partial
//      (m = its logit, l = 1, O = v_new).
//   1. cross-split log-sum-exp combine: global max M_h and sum L_h per query head,
//      out_h = (sum_p O_p 2^(m_p - M_h) + v_new 2^(s_new - M_h)) / L_h        (Eq. 2)
//   2. normalised probability of every decode token from the stored raw logits:
//      p = 2^(s - M_h) / L_h; mean over the G heads                           (Eq. 4)
//   3. I_i <- beta * I_i + abar_i; the fresh token starts from 0              (Eq. 5, 6)
//   4. overflow k = max(0, n - budget) (Eq. 7); the k smallest 64-bit keys
//      (fp32 score bits, position id) are the evicted set (Eq. 8).  Scores are
//      non-negative so their bit patterns order like the values: selection is integer
//      work on exactly the scores that are stored.  k = 1: arg-min reduction.
//      k > 1: 8-pass byte-wise radix select of the k-th key.
//   5. append + compaction (Eq. 9).  k = 0: the fresh row goes to slot n_old.  k = 1: the
//      fresh row goes straight into the evicted slot (nothing is written when the fresh
//      token itself is the one evicted), which leaves the pool exactly as "append at the
//      end, then move the last row into the hole" would.  k > 1: append, then survivors
//      stored beyond the new count move into the holes (K row, V row, score, position id).
//      Slot order changes, which is harmless: softmax and sum(p v) do not depend on the
//      order and ties are broken by position id.
// NT threads take part (a multiple of 32); they synchronise on named barrier BAR only,
// so a subset of a CTA can run the tail while other warps keep streaming.
#pragma once
#include "mkv_common.cuh"

namespace mkv {

template <int NT>
struct TailSmem {
    float M[kMaxGroup];
    float invL[kMaxGroup];
    float snew[kMaxGroup];   // logit of the fresh token (log2 units)
    float wnew[kMaxGroup];   // 2^(snew - M)
    float w[kMaxParts][kMaxGroup];    // running max of a partial, then its weight 2^(m - M)
    float pl[kMaxParts][kMaxGroup];   // running sum of a partial
    unsigned long long red_key[NT / 32];
    int red_slot[NT / 32];
    int hist[256];
    int cnt[3][NT / 32];
    int misc[4];
    int par;                 // parity of this launch: which copy of the unit counters is in use
};

__device__ inline void copy_row_swizzled(uint8_t* pool, size_t unit_base, int rowb, int src, int dst,
                                         int lane) {
    const int chunks = rowb >> 4;
    const uint4* s = reinterpret_cast<const uint4*>(pool + unit_base + (size_t)src * rowb);
    uint4* d = reinterpret_cast<uint4*>(pool + unit_base + (size_t)dst * rowb);
    for (int c = lane; c < chunks; c += 32) d[c ^ (dst & 7)] = __ldcg(&s[c ^ (src & 7)]);
}

// plain row (k_new / v_new of the unit) -> pool slot `dst`, chunk-permuted
__device__ inline void store_row_swizzled(uint8_t* pool, size_t unit_base, int rowb, const void* src_row, int dst,
                                          int lane) {
    const int chunks = rowb >> 4;
    const uint4* s = reinterpret_cast<const uint4*>(src_row);
    uint4* d = reinterpret_cast<uint4*>(pool + unit_base + (size_t)dst * rowb);
    for (int c = lane; c < chunks; c += 32) d[c ^ (dst & 7)] = __ldg(&s[c]);
}

// N consecutive elements of type T as floats, fetched with one vector load.
template <typename T, int N>
__device__ inline void load_elems(const T* ptr, float (&f)[N]) {
    static_assert(N == 2 || N == 4, "two or four elements");
    if constexpr (sizeof(T) * N == 16) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(ptr));
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < N; ++i) f[i] = to_f32(e[i]);
    } else if constexpr (sizeof(T) * N == 8) {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(ptr));
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < N; ++i) f[i] = to_f32(e[i]);
    } else {
        const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(ptr));
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < N; ++i) f[i] = to_f32(e[i]);
    }
}

// The unit is complete: prepare the idle copy of its counters for the next launch.
__device__ inline void rewind_unit(const LayerDev& L, int u, int par) {
    const int idle = (par ^ 1) * L.n_units + u;
    L.next[idle] = L.unit_next0[u];
    L.cnt[idle] = make_int2(0, 0);
}

// What a tail can fetch before its unit is complete (nothing here is written by the step
// until the tail itself runs): the unit's decode count and step number, the scores and
// position ids of the tokens this thread will handle in the first two passes, and the fresh
// token's value elements; the fresh token's logits go to shared memory.
template <int NT, int GB>
struct TailPre {
    static constexpr int TW = GB <= 4 ? 4 : 2;          // tokens per thread and pass (one 16- or 8-byte vector)
    static constexpr int OCB = (GB * 32 + NT - 1) / NT; // float4 output elements per thread (bound)
    int n_dec, t;
    float sc[2][TW];
    int ps[2][TW];
    float vn[OCB][4];
};

__device__ inline void store_out4(const Params& p, size_t idx, float4 v) {
    if (p.out_f32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + idx) = v;
    } else {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&lo);
        pk.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + idx) = pk;
    }
}

template <int TW>
__device__ inline void load_vec(const float* src, float (&dst)[TW]) {
    if constexpr (TW == 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(src));
        dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    } else {
        const float2 v = __ldcg(reinterpret_cast<const float2*>(src));
        dst[0] = v.x; dst[1] = v.y;
    }
}
template <int TW>
__device__ inline void load_vec(const int32_t* src, int (&dst)[TW]) {
    float f[TW];
    load_vec<TW>(reinterpret_cast<const float*>(src), f);
#pragma unroll
    for (int j = 0; j < TW; ++j) dst[j] = __float_as_int(f[j]);
}

// GB: compile-time bound of the group size G (4 or 8); it sizes the register staging.
// LAYER: the scores are updated later, for all KV heads of the sequence at once; none fetched here.
template <typename T, int NT, int GB, bool LAYER = false>
__device__ void tail_prefetch(const Params& p, int u, TailSmem<NT>& sm, int tid, TailPre<NT, GB>& pre) {
    constexpr int TW = TailPre<NT, GB>::TW, OCB = TailPre<NT, GB>::OCB, NW = NT / 32;
    const LayerDev& L = p.L;
    const int G = p.group, D = p.head_dim, ls = p.lstride;
    const int b = u / p.kv_heads, g = u - b * p.kv_heads;
    const int lane = tid & 31, warp = tid >> 5;
    const bool dec = (p.mode == kModeDecode);
    pre.n_dec = L.n_dec[u];
    pre.t = L.unit_step[u];
    if (!dec) return;
    const T* qrow = reinterpret_cast<const T*>(p.q) + ((size_t)b * p.q_heads + (size_t)g * G) * D;
    const T* knew = reinterpret_cast<const T*>(p.k_new) + (size_t)u * D;
    const T* vnew = reinterpret_cast<const T*>(p.v_new) + (size_t)u * D;
    const float* score = L.score + (size_t)u * ls;
    const int32_t* pos = L.pos + (size_t)u * ls;
    const int n_old = min(pre.n_dec, p.cap - 1);
    if constexpr (!LAYER) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int i0 = TW * (tid + k * NT);
            if (i0 < n_old) { load_vec<TW>(score + i0, pre.sc[k]); load_vec<TW>(pos + i0, pre.ps[k]); }
        }
    }
    const int ne = G * D / 4;
#pragma unroll
    for (int c = 0; c < OCB; ++c) {
        const int e = tid + c * NT;
        if (e < ne) load_elems<T, 4>(vnew + (4 * e) % D, pre.vn[c]);
    }
    // logit of the fresh token: lane l holds D/32 consecutive elements
    for (int h = warp; h < G; h += NW) {
        float a = 0.f;
        if (D == 128) {
            float qv[4], kv[4];
            load_elems<T, 4>(qrow + (size_t)h * D + 4 * lane, qv);
            load_elems<T, 4>(knew + 4 * lane, kv);
            a = fmaf(qv[0], kv[0], fmaf(qv[1], kv[1], fmaf(qv[2], kv[2], qv[3] * kv[3])));
        } else {
            float qv[2], kv[2];
            load_elems<T, 2>(qrow + (size_t)h * D + 2 * lane, qv);
            load_elems<T, 2>(knew + 2 * lane, kv);
            a = fmaf(qv[0], kv[0], qv[1] * kv[1]);
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        if (lane == 0) sm.snew[h] = a * p.scale_log2;
    }
}

// The tail proper; P = partial slots the unit's visits took.
// LAYER (score mode "mean over all heads of the layer"): the tail stops after `out` and the
// probabilities.  Per decode token it adds the SUM over the unit's G heads of the normalised
// probabilities (the fresh token's at index n_old) to the sequence's row of head sums (vector
// atomics; in the reproducible mode it stores them in a row of its own instead, and the rows
// are added up in KV-head order later); scores, selection and compaction follow for all KV
// heads of the sequence together (layer_finish).
template <typename T, int NT, int BAR, int GB, bool LAYER = false>
__device__ void unit_tail(const Params& p, int u, int P_in, const TailPre<NT, GB>& pre, TailSmem<NT>& sm, int tid) {
    const LayerDev& L = p.L;
    const int G = p.group, D = p.head_dim, cap = p.cap, ls = p.lstride;
    const int rowb = D * (int)sizeof(T);
    const int b = u / p.kv_heads, g = u - b * p.kv_heads;
    const int P = min(P_in, kMaxParts), part0 = u * kMaxParts;
    const bool dec = (p.mode == kModeDecode);
    const int n_old = min(pre.n_dec, dec ? cap - 1 : cap);
    const int n = dec ? n_old + 1 : n_old;
    const int t = pre.t;
    const int lane = tid & 31, warp = tid >> 5;
    constexpr int NW = NT / 32;
    constexpr int TW = TailPre<NT, GB>::TW;
    constexpr int PB = GB <= 4 ? 4 : 1;                 // partials staged in registers up front
    constexpr int LB = 4;                               // partials fetched per trip after those
    constexpr int OCB = TailPre<NT, GB>::OCB;
    const T* knew = reinterpret_cast<const T*>(p.k_new) + (size_t)u * D;
    const T* vnew = reinterpret_cast<const T*>(p.v_new) + (size_t)u * D;
    float* score = L.score + (size_t)u * ls;
    int32_t* pos = L.pos + (size_t)u * ls;
    const float* lg = L.logit + ((size_t)b * p.q_heads + (size_t)g * G) * ls;
    float* psum = L.head_sum + (size_t)b * ls;                              // LAYER only
    float* usum = L.unit_sum + (size_t)u * ls;                              // LAYER, reproducible mode
    const float* po_base = L.part_o + (size_t)part0 * G * D;
    const size_t pstride = (size_t)G * D;
    const int ne = G * D / 4;                           // float4 elements of one partial / of `out`
    if (tid == 0) MKV_TR(8);

    // Everything below is latency: a few dependent trips to L2.  So every load that does
    // not need the softmax statistics is issued first, in one batch: the logits of this
    // thread's tokens (first two passes), its share of the first partials' O, and the
    // partials' (m, l).
    struct Tok { float lgv[GB][TW]; };
    auto load_tok = [&](int i0, Tok& r) {
        if (i0 < n_old) {
#pragma unroll
            for (int h = 0; h < GB; ++h)
                if (h < G) load_vec<TW>(lg + (size_t)h * ls + i0, r.lgv[h]);
        }
    };
    Tok tk;
    if (dec) load_tok(TW * tid, tk);
    float4 po[PB][OCB];
#pragma unroll
    for (int q = 0; q < PB; ++q)
#pragma unroll
        for (int c = 0; c < OCB; ++c) {
            const int e = tid + c * NT;
            po[q][c] = (q < P && e < ne) ? __ldcg(reinterpret_cast<const float4*>(po_base + (size_t)q * pstride) + e)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    for (int e0 = 0; e0 < P * kMaxGroup; e0 += NT) {
        const int e = e0 + tid, q = e / kMaxGroup, h = e - q * kMaxGroup;
        if (q < P && h < G) {
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(&L.part_ml[((size_t)(part0 + q) * G + h) * 2]));
            sm.w[q][h] = ml.x;
            sm.pl[q][h] = ml.y;
        }
    }
    if (tid == 0) MKV_TR(9);
    bar_sync(BAR, NT);
    if (tid == 0) MKV_TR(10);

    // ---- 1. combine -----------------------------------------------------------------------
    // heads over the warps, partials over the lanes (two per lane: kMaxParts = 64)
    static_assert(kMaxParts <= 64, "two partials per lane");
    for (int h = warp; h < G; h += NW) {
        const bool has0 = lane < P, has1 = lane + 32 < P;
        const float m0 = has0 ? sm.w[lane][h] : kNegBig;
        const float m1 = has1 ? sm.w[lane + 32][h] : kNegBig;
        float M = fmaxf(m0, m1);
        if (dec) M = fmaxf(M, sm.snew[h]);
#pragma unroll
        for (int off = 16; off; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
        const float w0 = has0 ? fast_exp2(m0 - M) : 0.f;
        const float w1 = has1 ? fast_exp2(m1 - M) : 0.f;
        float Lsum = (has0 ? sm.pl[lane][h] * w0 : 0.f) + (has1 ? sm.pl[lane + 32][h] * w1 : 0.f);
#pragma unroll
        for (int off = 16; off; off >>= 1) Lsum += __shfl_xor_sync(0xffffffffu, Lsum, off);
        if (has0) sm.w[lane][h] = w0;
        if (has1) sm.w[lane + 32][h] = w1;
        if (lane == 0) {
            float wn = 0.f;
            if (dec) { wn = fast_exp2(sm.snew[h] - M); Lsum += wn; }
            sm.wnew[h] = wn;
            sm.M[h] = M;
            sm.invL[h] = Lsum > 0.f ? 1.0f / Lsum : 0.f;
        }
    }
    bar_sync(BAR, NT);
    // out, part 1: the fresh token and the partials staged in registers
    const size_t obase = ((size_t)b * p.q_heads + (size_t)g * G) * D;
    float4 oacc[OCB];
#pragma unroll
    for (int c = 0; c < OCB; ++c) {
        const int e = tid + c * NT;
        const int h = min((4 * e) / D, G - 1);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (dec) {
            const float wn = sm.wnew[h];
            acc = make_float4(pre.vn[c][0] * wn, pre.vn[c][1] * wn, pre.vn[c][2] * wn, pre.vn[c][3] * wn);
        }
#pragma unroll
        for (int q = 0; q < PB; ++q) {
            if (q < P) {
                const float w = sm.w[q][h];
                acc.x = fmaf(po[q][c].x, w, acc.x); acc.y = fmaf(po[q][c].y, w, acc.y);
                acc.z = fmaf(po[q][c].z, w, acc.z); acc.w = fmaf(po[q][c].w, w, acc.w);
            }
        }
        oacc[c] = acc;
    }
    // out, part 2: the remaining partials, several per trip, then the store
    auto finish_out = [&]() {
#pragma unroll
        for (int c = 0; c < OCB; ++c) {
            const int e = tid + c * NT;
            if (e >= ne) continue;
            const int h = (4 * e) / D;
            float4 acc = oacc[c];
            for (int q0 = PB; q0 < P; q0 += LB) {
                float4 v[LB];
#pragma unroll
                for (int j = 0; j < LB; ++j)
                    v[j] = (q0 + j < P) ? __ldcg(reinterpret_cast<const float4*>(po_base + (size_t)(q0 + j) * pstride) + e)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < LB; ++j) {
                    const float w = (q0 + j < P) ? sm.w[q0 + j][h] : 0.f;
                    acc.x = fmaf(v[j].x, w, acc.x); acc.y = fmaf(v[j].y, w, acc.y);
                    acc.z = fmaf(v[j].z, w, acc.z); acc.w = fmaf(v[j].w, w, acc.w);
                }
            }
            const float il = sm.invL[h];
            store_out4(p, obase + 4 * (size_t)e, make_float4(acc.x * il, acc.y * il, acc.z * il, acc.w * il));
        }
    };
    if (!dec) {
        finish_out();
        if (tid == 0) MKV_TR(11);
        if (tid == 0) rewind_unit(L, u, sm.par);
        return;
    }
    if (tid == 0) MKV_TR(11);

    // ---- 2./3. probabilities, head mean, momentum update ---------------------------------
    const int k = max(0, n - p.budget);
    const float inv_g = 1.0f / (float)G;
    unsigned long long* keys = L.keys + (size_t)u * cap;
    float sum_new = 0.f;
    for (int h = 0; h < G; ++h) sum_new = fmaf(sm.wnew[h], sm.invL[h], sum_new);
    const float ab_new = sum_new * inv_g;             // Eq. 6: I_fresh = alpha * 0 + abar_fresh
    const unsigned long long key_new = ((unsigned long long)__float_as_uint(ab_new) << 32) | (unsigned)t;
    unsigned long long best_key = ~0ull;
    int best_slot = -1;
    auto process_tok = [&](int i0, const Tok& r, const float (&sc)[TW], const int (&ps)[TW]) {
        if (i0 >= n_old) return;
        float ab[TW], nw[TW];
#pragma unroll
        for (int j = 0; j < TW; ++j) ab[j] = 0.f;
#pragma unroll
        for (int h = 0; h < GB; ++h) {
            if (h < G) {
                const float Mh = sm.M[h], iLh = sm.invL[h];
#pragma unroll
                for (int j = 0; j < TW; ++j) ab[j] = fmaf(fast_exp2(r.lgv[h][j] - Mh), iLh, ab[j]);
            }
        }
        if constexpr (LAYER) {
            if (p.det) {
#pragma unroll
                for (int j = 0; j < TW; ++j) if (i0 + j < n_old) usum[i0 + j] = ab[j];
            } else if (i0 + TW <= n_old) {
                if constexpr (TW == 4) atomicAdd(reinterpret_cast<float4*>(psum + i0), make_float4(ab[0], ab[1], ab[2], ab[3]));
                else atomicAdd(reinterpret_cast<float2*>(psum + i0), make_float2(ab[0], ab[1]));
            } else {
#pragma unroll
                for (int j = 0; j < TW; ++j) if (i0 + j < n_old) atomicAdd(psum + i0 + j, ab[j]);
            }
            return;
        }
#pragma unroll
        for (int j = 0; j < TW; ++j) {
            ab[j] *= inv_g;
            nw[j] = fmaf(p.beta, sc[j], ab[j]);
        }
        if (i0 + TW <= n_old) {
            if constexpr (TW == 4) *reinterpret_cast<float4*>(score + i0) = make_float4(nw[0], nw[1], nw[2], nw[3]);
            else *reinterpret_cast<float2*>(score + i0) = make_float2(nw[0], nw[1]);
        } else {
#pragma unroll
            for (int j = 0; j < TW; ++j) if (i0 + j < n_old) score[i0 + j] = nw[j];
        }
#pragma unroll
        for (int j = 0; j < TW; ++j) {
            if (i0 + j < n_old) {
                if (L.abar) { L.abar[(size_t)u * cap + i0 + j] = ab[j]; L.abar_pos[(size_t)u * cap + i0 + j] = ps[j]; }
                const unsigned long long key = ((unsigned long long)__float_as_uint(nw[j]) << 32) | (unsigned)ps[j];
                if (k > 1) keys[i0 + j] = key;
                if (key < best_key) { best_key = key; best_slot = i0 + j; }
            }
        }
    };
    process_tok(TW * tid, tk, pre.sc[0], pre.ps[0]);
    // further passes; the rest of `out` travels with the first of them (one trip, not two)
    bool out_done = false;
    for (int base = TW * NT, pass = 1; base < n_old; base += TW * NT, ++pass) {
        const int i0 = base + TW * tid;
        load_tok(i0, tk);
        float sc[TW];
        int ps[TW];
        if (pass == 1) {
#pragma unroll
            for (int j = 0; j < TW; ++j) { sc[j] = pre.sc[1][j]; ps[j] = pre.ps[1][j]; }
        } else if (!LAYER && i0 < n_old) {
            load_vec<TW>(score + i0, sc);
            load_vec<TW>(pos + i0, ps);
        }
        if (!out_done) { finish_out(); out_done = true; }
        process_tok(i0, tk, sc, ps);
    }
    if (!out_done) finish_out();
    if (tid == 0) MKV_TR(12);
    if constexpr (LAYER) {
        if (tid == NT - 1) {
            if (p.det) usum[n_old] = sum_new;
            else atomicAdd(psum + n_old, sum_new);
        }
        return;
    }
    if (tid == NT - 1) {                              // the fresh token sits (virtually) in slot n_old
        if (key_new < best_key) { best_key = key_new; best_slot = n_old; }
        if (L.abar) { L.abar[(size_t)u * cap + n_old] = ab_new; L.abar_pos[(size_t)u * cap + n_old] = t; }
    }
    if (tid == 0) { L.n_prev[u] = n; L.ev_k[u] = k; L.n_dec[u] = n - k; L.unit_step[u] = t + 1; }

    const size_t ubase = (size_t)u * cap * rowb;
    if (k != 1) {
        // ---- 5 (k = 0, and first half of k > 1): append at the end ----------------------
        if (warp == 0) store_row_swizzled(L.Kd, ubase, rowb, knew, n_old, lane);
        if (warp == (NW > 1 ? 1 : 0)) store_row_swizzled(L.Vd, ubase, rowb, vnew, n_old, lane);
        if (tid == NT - 1) { score[n_old] = ab_new; pos[n_old] = t; keys[n_old] = key_new; }
        if (k == 0) {
            if (tid == 0) rewind_unit(L, u, sm.par);
            return;
        }
    }

    if (k == 1) {
        // ---- 4a. arg-min over (score bits, position id) ------------------------------
        for (int off = 16; off; off >>= 1) {
            const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best_key, off);
            const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
            if (ok < best_key) { best_key = ok; best_slot = os; }
        }
        if (lane == 0) { sm.red_key[warp] = best_key; sm.red_slot[warp] = best_slot; }
        if (tid == 0) MKV_TR(14);
        if (tid == NT - 1) MKV_TR(15);
        bar_sync(BAR, NT);   // also orders every score write before the stores below
        unsigned long long kk = sm.red_key[0];
        int e = sm.red_slot[0];
        for (int w2 = 1; w2 < NW; ++w2)
            if (sm.red_key[w2] < kk) { kk = sm.red_key[w2]; e = sm.red_slot[w2]; }
        if (tid == 0) {
            L.ev_pos[(size_t)u * cap] = (int32_t)(unsigned)(kk & 0xffffffffu);
            L.ev_score[(size_t)u * cap] = __uint_as_float((unsigned)(kk >> 32));
        }
        if (tid == 0) MKV_TR(13);
        // ---- 5a. the fresh row lands in the hole -----------------------------------------
        if (e != n_old) {
            if (warp == 0) store_row_swizzled(L.Kd, ubase, rowb, knew, e, lane);
            if (warp == (NW > 1 ? 1 : 0)) store_row_swizzled(L.Vd, ubase, rowb, vnew, e, lane);
            if (tid == NT - 1) { score[e] = ab_new; pos[e] = t; }
        }
        if (tid == 0) rewind_unit(L, u, sm.par);
        return;
    }

    // ---- 4b. radix select of the k-th smallest key (keys are distinct) ----------------
    bar_sync(BAR, NT);       // keys, scores and the appended row are in place
    unsigned long long prefix = 0ull, mask = 0ull;
    int want = k - 1;
    for (int pass = 7; pass >= 0; --pass) {
        for (int i = tid; i < 256; i += NT) sm.hist[i] = 0;
        bar_sync(BAR, NT);
        for (int i = tid; i < n; i += NT) {
            const unsigned long long key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&sm.hist[(int)((key >> (8 * pass)) & 255ull)], 1);
        }
        bar_sync(BAR, NT);
        if (tid == 0) {
            int cum = 0, sel = 255;
            for (int bin = 0; bin < 256; ++bin) {
                const int c = sm.hist[bin];
                if (want < cum + c) { sel = bin; break; }
                cum += c;
            }
            sm.misc[0] = sel;
            sm.misc[1] = want - cum;
        }
        bar_sync(BAR, NT);
        prefix |= (unsigned long long)sm.misc[0] << (8 * pass);
        mask |= 255ull << (8 * pass);
        want = sm.misc[1];
    }
    const unsigned long long kth = prefix;

    // ---- 5b. ordered lists of holes (< n') and movers (>= n'), then the moves ---------
    const int n_new = n - k;
    int32_t* holes = L.list_a + (size_t)u * cap;
    int32_t* movers = L.list_b + (size_t)u * cap;
    int hc = 0, mc = 0, ec = 0;
    for (int base = 0; base < n; base += NT) {
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
        if (lane == 0) { sm.cnt[0][warp] = __popc(bh); sm.cnt[1][warp] = __popc(bm); sm.cnt[2][warp] = __popc(be); }
        bar_sync(BAR, NT);
        int ph = 0, pm = 0, pe = 0, th = 0, tm = 0, te = 0;
        for (int w2 = 0; w2 < NW; ++w2) {
            if (w2 < warp) { ph += sm.cnt[0][w2]; pm += sm.cnt[1][w2]; pe += sm.cnt[2][w2]; }
            th += sm.cnt[0][w2]; tm += sm.cnt[1][w2]; te += sm.cnt[2][w2];
        }
        if (hole) holes[hc + ph + __popc(bh & lt)] = i;
        if (mover) movers[mc + pm + __popc(bm & lt)] = i;
        if (ev) {
            const int j = ec + pe + __popc(be & lt);
            L.ev_pos[(size_t)u * cap + j] = (int32_t)(unsigned)(key & 0xffffffffu);
            L.ev_score[(size_t)u * cap + j] = __uint_as_float((unsigned)(key >> 32));
        }
        hc += th; mc += tm; ec += te;
        bar_sync(BAR, NT);
    }
    if (hc != mc || ec != k) {
        if (tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
    } else {
        for (int j = warp; j < hc; j += NW) {
            const int src = movers[j], dst = holes[j];
            copy_row_swizzled(L.Kd, ubase, rowb, src, dst, lane);
            copy_row_swizzled(L.Vd, ubase, rowb, src, dst, lane);
            if (lane == 0) { score[dst] = score[src]; pos[dst] = pos[src]; }
        }
    }
    if (tid == 0) rewind_unit(L, u, sm.par);
}

}  // namespace mkv
