// Scoring exactly as Eq. 4 prints it: the attention a decode token receives is averaged over
// ALL H query heads of the layer, the layer keeps ONE importance vector per sequence, and all
// KV heads evict the same tokens (score mode MKV_SCORE_LAYER_MEAN with more than one KV
// head).  The streaming loops run unchanged.  When a (sequence, KV head) unit is complete its
// tail does that head's share (unit_tail in its LAYER form):
//   the fresh token's logits, the cross-split combine, `out`                        (Eq. 2)
//   per decode token the sum over the unit's G heads of 2^(s - M_h) / L_h, added to the
//   sequence's row of head sums
// and the tail that finishes last for a sequence (a ticket) goes on with what needs all heads
// (layer_finish, this file):
//   per decode token: abar = (1/H) of the summed probabilities of all H heads         (Eq. 4)
//   I <- beta * I + abar, the fresh token starting from 0                            (Eq. 5, 6)
//   one selection of the overflow-many lowest (score bits, position id) keys         (Eq. 7, 8)
//   the same append / hole filling in every KV head's pool                           (Eq. 9)
// Every KV head's unit holds an equal copy of the scores, position ids and counts, so the
// streaming loops and the inspection calls need not know about the mode.  Nothing of a
// sequence's pools, counts or scores is written before all its units are complete, so units of
// the sequence that are still being streamed see the step's input state.
// NT threads take part (a multiple of 32) and synchronise on named barrier BAR only.
#pragma once
#include "mkv_tail.cuh"

namespace mkv {

template <typename T, int NT, int BAR, int GB>
__device__ void layer_finish(const Params& p, int u, const TailPre<NT, GB>& pre, TailSmem<NT>& sm, int tid) {
    constexpr int NW = NT / 32;
    constexpr int TW = TailPre<NT, GB>::TW;            // tokens per thread and pass
    const LayerDev& L = p.L;
    const int lane = tid & 31, warp = tid >> 5;
    const int G = p.group, D = p.head_dim, cap = p.cap, ls = p.lstride, Hkv = p.kv_heads, Hq = p.q_heads;
    const int rowb = D * (int)sizeof(T);
    const int b = u / Hkv, u0 = b * Hkv;
    const int par = sm.par;

    // The unit's sums are written: take a ticket.  The tail that draws the last one of the
    // sequence goes on (and leaves the ticket at zero for the next step).
    __threadfence();
    bar_sync(BAR, NT);
    if (tid == 0) {
        const int last = (atomicAdd(&L.seq_ticket[b], 1) == Hkv - 1);
        if (last) L.seq_ticket[b] = 0;
        sm.misc[2] = last;
    }
    bar_sync(BAR, NT);
    const bool last = sm.misc[2] != 0;
    bar_sync(BAR, NT);          // everyone has read the flag before a later tail writes it again
    if (!last) return;
    __threadfence();

    const int n_old = min(pre.n_dec, cap - 1);         // (equal in every unit of the sequence)
    const int n = n_old + 1;
    const int t = pre.t;
    const int k = max(0, n - p.budget);
    // the sequence's head sums, complete now; this tail reads them and leaves the row at zero
    float* const sums = L.head_sum + (size_t)b * ls;

    // ---- all heads: head mean, momentum update -----------------------------------------------
    const float inv_h = 1.0f / (float)Hq;
    // (reproducible mode: every unit kept its own row of sums; they are added in KV-head order)
    const float* const usums = L.unit_sum + (size_t)u0 * ls;
    auto load_sums = [&](int i, float (&dst)[TW]) {
        if (!p.det) { load_vec<TW>(sums + i, dst); return; }
#pragma unroll
        for (int j = 0; j < TW; ++j) dst[j] = 0.f;
        for (int g2 = 0; g2 < Hkv; ++g2) {
            float part[TW];
            load_vec<TW>(usums + (size_t)g2 * ls + i, part);
#pragma unroll
            for (int j = 0; j < TW; ++j) dst[j] += part[j];
        }
    };
    float sum_fresh = 0.f;
    if (p.det) { for (int g2 = 0; g2 < Hkv; ++g2) sum_fresh += __ldcg(usums + (size_t)g2 * ls + n_old); }
    else sum_fresh = __ldcg(sums + n_old);
    const float ab_new = sum_fresh * inv_h;                // Eq. 6: I_fresh = alpha * 0 + abar_fresh
    const unsigned long long key_new = ((unsigned long long)__float_as_uint(ab_new) << 32) | (unsigned)t;
    unsigned long long* keys = L.keys + (size_t)u0 * cap;
    const float* score0 = L.score + (size_t)u0 * ls;
    const int32_t* pos0 = L.pos + (size_t)u0 * ls;
    unsigned long long best_key = ~0ull;
    int best_slot = -1;
    // TW tokens per thread and pass, two passes per trip: their loads are issued together (rows
    // are lstride floats long, a multiple of 4, so whole vectors stay inside them)
    auto token_pass = [&](int i0, const float (&s)[TW], const float (&sc)[TW], const int (&ps)[TW]) {
        if (i0 >= n_old) return;
        float ab[TW], nw[TW];
#pragma unroll
        for (int j = 0; j < TW; ++j) { ab[j] = s[j] * inv_h; nw[j] = fmaf(p.beta, sc[j], ab[j]); }
        const bool whole = i0 + TW <= n_old;
        // slots below n_old go back to zero (slot n_old, which every thread reads above, later)
        if (whole) {
            if constexpr (TW == 4) *reinterpret_cast<float4*>(sums + i0) = make_float4(0.f, 0.f, 0.f, 0.f);
            else *reinterpret_cast<float2*>(sums + i0) = make_float2(0.f, 0.f);
        } else {
            for (int j = 0; j < TW; ++j) if (i0 + j < n_old) sums[i0 + j] = 0.f;
        }
        for (int g2 = 0; g2 < Hkv; ++g2) {
            float* sg = L.score + (size_t)(u0 + g2) * ls + i0;
            if (whole) {
                if constexpr (TW == 4) *reinterpret_cast<float4*>(sg) = make_float4(nw[0], nw[1], nw[2], nw[3]);
                else *reinterpret_cast<float2*>(sg) = make_float2(nw[0], nw[1]);
            } else {
                for (int j = 0; j < TW; ++j) if (i0 + j < n_old) sg[j] = nw[j];
            }
            if (L.abar)
                for (int j = 0; j < TW; ++j)
                    if (i0 + j < n_old) {
                        L.abar[(size_t)(u0 + g2) * cap + i0 + j] = ab[j];
                        L.abar_pos[(size_t)(u0 + g2) * cap + i0 + j] = ps[j];
                    }
        }
#pragma unroll
        for (int j = 0; j < TW; ++j) {
            if (i0 + j < n_old) {
                const unsigned long long key = ((unsigned long long)__float_as_uint(nw[j]) << 32) | (unsigned)ps[j];
                if (k > 1) keys[i0 + j] = key;
                if (key < best_key) { best_key = key; best_slot = i0 + j; }
            }
        }
    };
    for (int base = 0; base < n_old; base += 2 * TW * NT) {
        const int ia = base + TW * tid, ib = ia + TW * NT;
        float sa[TW], sca[TW], sb[TW], scb[TW];
        int psa[TW], psb[TW];
        if (ia < n_old) { load_sums(ia, sa); load_vec<TW>(score0 + ia, sca); load_vec<TW>(pos0 + ia, psa); }
        if (ib < n_old) { load_sums(ib, sb); load_vec<TW>(score0 + ib, scb); load_vec<TW>(pos0 + ib, psb); }
        token_pass(ia, sa, sca, psa);
        token_pass(ib, sb, scb, psb);
    }
    bar_sync(BAR, NT);                                 // every thread has read slot n_old
    if (tid == NT - 1) {                               // the fresh token sits (virtually) in slot n_old
        sums[n_old] = 0.f;
        if (key_new < best_key) { best_key = key_new; best_slot = n_old; }
        if (L.abar)
            for (int g2 = 0; g2 < Hkv; ++g2) {
                L.abar[(size_t)(u0 + g2) * cap + n_old] = ab_new;
                L.abar_pos[(size_t)(u0 + g2) * cap + n_old] = t;
            }
    }
    for (int g2 = tid; g2 < Hkv; g2 += NT) {
        const int u2 = u0 + g2;
        L.n_prev[u2] = n; L.ev_k[u2] = k; L.n_dec[u2] = n - k; L.unit_step[u2] = t + 1;
        rewind_unit(L, u2, par);
    }

    // the fresh row of every KV head into slot `dst` of its pool, with the shared score and id
    auto place_fresh = [&](int dst) {
        for (int j = warp; j < 2 * Hkv; j += NW) {
            const int u2 = u0 + (j >> 1);
            const size_t ubase = (size_t)u2 * cap * rowb;
            if (j & 1) store_row_swizzled(L.Vd, ubase, rowb, reinterpret_cast<const T*>(p.v_new) + (size_t)u2 * D, dst, lane);
            else store_row_swizzled(L.Kd, ubase, rowb, reinterpret_cast<const T*>(p.k_new) + (size_t)u2 * D, dst, lane);
        }
        for (int g2 = tid; g2 < Hkv; g2 += NT) {
            L.score[(size_t)(u0 + g2) * ls + dst] = ab_new;
            L.pos[(size_t)(u0 + g2) * ls + dst] = t;
        }
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
        if (lane == 0) { sm.red_key[warp] = best_key; sm.red_slot[warp] = best_slot; }
        bar_sync(BAR, NT);   // also orders every score write before the stores below
        unsigned long long kk = sm.red_key[0];
        int e = sm.red_slot[0];
        for (int w2 = 1; w2 < NW; ++w2)
            if (sm.red_key[w2] < kk) { kk = sm.red_key[w2]; e = sm.red_slot[w2]; }
        for (int g2 = tid; g2 < Hkv; g2 += NT) {
            L.ev_pos[(size_t)(u0 + g2) * cap] = (int32_t)(unsigned)(kk & 0xffffffffu);
            L.ev_score[(size_t)(u0 + g2) * cap] = __uint_as_float((unsigned)(kk >> 32));
        }
        if (e != n_old) place_fresh(e);                // the fresh row lands in the hole
        bar_sync(BAR, NT);   // the reduction slots are free again for a later tail
        return;
    }

    // ---- overflow > 1: radix select of the k-th smallest key, then ordered hole filling ---------
    bar_sync(BAR, NT);
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
    const int n_new = n - k;
    int32_t* holes = L.list_a + (size_t)u0 * cap;
    int32_t* movers = L.list_b + (size_t)u0 * cap;
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
            for (int g2 = 0; g2 < Hkv; ++g2) {
                L.ev_pos[(size_t)(u0 + g2) * cap + j] = (int32_t)(unsigned)(key & 0xffffffffu);
                L.ev_score[(size_t)(u0 + g2) * cap + j] = __uint_as_float((unsigned)(key >> 32));
            }
        }
        hc += th; mc += tm; ec += te;
        bar_sync(BAR, NT);
    }
    if (hc != mc || ec != k) {
        if (tid == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
        return;
    }
    for (int j = warp; j < hc * Hkv; j += NW) {
        const int g2 = j / hc, m = j - g2 * hc;
        const int src = movers[m], dst = holes[m];
        const int u2 = u0 + g2;
        const size_t ubase = (size_t)u2 * cap * rowb;
        copy_row_swizzled(L.Kd, ubase, rowb, src, dst, lane);
        copy_row_swizzled(L.Vd, ubase, rowb, src, dst, lane);
        if (lane == 0) {
            L.score[(size_t)u2 * ls + dst] = L.score[(size_t)u2 * ls + src];
            L.pos[(size_t)u2 * ls + dst] = L.pos[(size_t)u2 * ls + src];
        }
    }
}

// The whole tail of a unit in this score mode.  GB as in unit_tail.
template <typename T, int NT, int BAR, int GB>
__device__ void layer_unit_tail(const Params& p, int u, int P_in, const TailPre<NT, GB>& pre, TailSmem<NT>& sm,
                                int tid) {
    unit_tail<T, NT, BAR, GB, true>(p, u, P_in, pre, sm, tid);
    layer_finish<T, NT, BAR, GB>(p, u, pre, sm, tid);
}

}  // namespace mkv
