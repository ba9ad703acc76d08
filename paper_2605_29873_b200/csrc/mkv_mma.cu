// Tensor-core split-KV decode attention for bf16 caches, head_dim 128, G <= 8: the hot
// path of the Llama-3.1-8B- and Qwen2.5-7B-shaped workloads.
//
// Decode attention at GQA group 4-7 is bound by streaming K and V from HBM once per KV
// head; the kernel is built around that stream.  A CTA is four kinds of warps:
//
//   * one PRODUCER thread pulls chunks of 64-row tiles from per-unit atomic counters,
//     starting at the CTA's own place and moving on to the next unit with tiles left when
//     its unit is exhausted, and issues bulk asynchronous copies (the
//     non-tensor TMA form, no multicast) of K and V tiles, 16 KB each, into a ring of
//     shared-memory stages; completion is signalled on an mbarrier (complete_tx).  The
//     cache rows are already chunk-permuted in HBM, so a straight copy lands a layout that
//     ldmatrix reads without bank conflicts.  At the start of a unit visit it also copies
//     the unit's G query rows into one of two small query slots.  The producer runs ahead
//     across unit boundaries.
//   * four CONSUMER warps each own 16 rows of a tile and never synchronise with one
//     another.  S = Q K^T uses mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the G
//     query heads in the M dimension; its accumulator fragment is, register for register,
//     the B operand of the transposed second product O^T += V^T P^T (head_dim in M, the
//     heads in N = 8), so P never leaves the registers and no work is spent on padding
//     rows.  This is not a GEMM reshaping for the sake of tensor cores: it takes the
//     per-row instruction count from ~60 (scalar FMA + shuffles) to ~4 so that issue slots
//     never limit the HBM stream, for G = 7 as well as G = 4.  The softmax runs in
//     registers in fp32 (quad shuffles for the row maximum); P enters the second mma as
//     hi + lo bf16 halves, so the rounding of P to bf16 does not reach `out`.
//     Raw fp32 logits of decode-pool tokens are stored (4 bytes per head and token) for
//     the tail, which needs the global log-sum-exp before it can normalise them (Eq. 4).
//   * one MERGE warp.  At the end of a unit visit the consumers drop their (m, l, O) into a
//     ring stage borrowed from the producer and go straight on to the next unit; the merge
//     warp folds the four states into one partial in global memory, returns the stage, adds
//     the visit's tiles to the unit's count.
//   * four TAIL warps, which watch the counts of the units this CTA looks after (the ones it starts
//     in) and run a
//     unit's tail (fresh token, combine, probabilities, momentum update, selection,
//     append/compaction) as soon as its count is complete, while the stream continues.
//     (Handing a completed unit to the CTA that delivered its last tiles instead, with a queue
//     for the overflow, lets CTAs leave earlier but serialises the tails of the units that
//     complete last on the few CTAs still running: 41.6 against 39.1 us per headline step.)
// Every wait is bounded (the context's wait limit): on expiry the kernel records
// MKV_ERR_TIMEOUT, every role drains (the producer waits, bounded again, for its copies in
// flight) and the CTA returns.
//
// CTAs wait on one another (a unit's tail waits for tiles other CTAs deliver), so the whole
// grid has to be resident at once: the host sizes it from the occupancy the device reports.
//
// Two optional behaviours, both decided by the context:
//   * early inputs: the caller's q is final when the launch is enqueued, so the consumers may
//     work through the CTA's reserved prompt tiles (frozen rows) while the previous kernel of
//     the stream is still running its last tails; everything else waits for it as usual.
//     When, on top of that, the previous kernel worked on other layers (the host knows), the
//     launch shares nothing with it -- layers are independent instances of Algorithm 1 and the
//     step scratch exists twice -- and is "deferred": no role waits at the start, CTAs stream as
//     soon as they get an SM, and the dependency wait is left to the first tail thread, which has
//     nothing to do until the first unit completes: it returns when the previous kernel has
//     ended, and only then does the CTA allow the next launch to begin (whose CTAs take the SMs
//     of this launch's CTAs as they finish).  At most two launches are ever in flight and they
//     complete in stream order.
//   * reproducible mode: no counters; every CTA covers a fixed range of the global tile
//     sequence and delivers a fixed partial slot, so the same inputs give the same bits.
#include "mkv_launch.h"
#include "mkv_ptx.cuh"
#include "mkv_layer_tail.cuh"
#include "mkv_tail.cuh"

namespace mkv {
namespace {

constexpr int kRowB = 256;                                // 128 bf16
constexpr int kTileBytes = kTileRows * kRowB;             // 16 KB (K or V)
constexpr int kStageBytes = 2 * kTileBytes;               // K then V
constexpr int kQRowB = kRowB + 16;                         // padded query row: the heads fall into different banks
constexpr int kQSlotBytes = kMaxGroup * kQRowB;           // query rows of one unit
constexpr int kQSlots = 2;
constexpr int kConsumerWarps = 4;
constexpr int kTailWarps = 4;
constexpr int kTailThreads = kTailWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;             // warp 4
constexpr int kMergeWarp = kConsumerWarps + 1;            // warp 5
constexpr int kTailTid0 = (kMergeWarp + 1) * 32;          // first thread of the tail group
constexpr int kThreads = kTailTid0 + kTailThreads;
constexpr int kMaxStages = 8;
constexpr int kXoStride = 132;                            // floats per head row of the exchange
constexpr size_t kSmemPerCta = 232448;                    // opt-in shared memory of one CTA on sm_100

enum : int { kEntryTile = 0, kEntryExchange = 1, kEntryEnd = 2 };

struct StageMeta {
    int kind;
    int unit;
    int seg;        // 0 prefill, 1 decode
    int row;        // slot of the tile's first row inside its pool (multiple of 64)
    int cnt;        // valid rows
    int first;      // first entry of a unit visit: reset the running state
    int slot;       // exchange entries: the visit's partial slot ...
    int ntiles;     // ... the tiles it covered ...
    int total;      // ... and the unit's tile count
    int pre;        // issued before the dependency wait: touches nothing an earlier kernel writes
};

struct ExchangeRef { int stage, unit, slot, ntiles, total; };   // stage < 0: no more exchanges

struct Control {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    unsigned long long xfull[kMaxStages];
    unsigned long long qfull[kQSlots];
    unsigned long long qempty[kQSlots];
    StageMeta meta[kMaxStages];
    ExchangeRef xq[kMaxStages];
    int abort_flag;
    int tail_unit;     // the unit whose tail the group runs next, or -1: leave
    int par;           // parity of this launch (the producer finds it after the dependency wait); -1 before
};

constexpr size_t smem_bytes(int nst) {
    return (size_t)nst * kStageBytes + kQSlots * kQSlotBytes + sizeof(TailSmem<kTailThreads>) + sizeof(Control) + 64;
}

__device__ inline bool aborted(const Control* ctl) { return *reinterpret_cast<const volatile int*>(&ctl->abort_flag) != 0; }

__device__ inline void note_timeout(const Params& p, Control* ctl) {
    atomicCAS(p.status, kStatusOk, kStatusTimeout);
    *reinterpret_cast<volatile int*>(&ctl->abort_flag) = 1;
}

// Bounded mbarrier wait that also gives up as soon as another role has aborted.
__device__ inline bool wait_or_abort(uint32_t bar, uint32_t parity, Control* ctl, unsigned long long limit_ns) {
    for (int i = 0; i < 32; ++i)
        if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (ptx::mbar_try_wait(bar, parity)) return true;
        if (aborted(ctl)) return false;
        if (ptx::globaltimer_ns() - t0 > limit_ns) return false;
    }
}

// The two counts of a unit live in one 8-byte word (tiles delivered in the low half, partial
// slots taken in the high half), which the unit's tail reads with one load; they are only ever
// changed by 8-byte atomics on the whole word.
__device__ inline unsigned long long count_add(int2* cnt, unsigned long long v) {
    return atomicAdd(reinterpret_cast<unsigned long long*>(cnt), v);
}

// The tail warps' loop over the units this CTA looks after.  While a unit is still being
// streamed the group already fetches what its tail needs and the step does not change
// (tail_prefetch); thread 0 then watches the unit's counters, which arrive as one 8-byte
// word (tiles delivered, partial slots taken).
// LAYER: the tails of a sequence's KV heads score together (Eq. 4 over all heads of the layer).
template <int GB, bool LAYER>
__device__ void tail_group(const Params& p, Control* ctl, TailSmem<kTailThreads>* tsm, int tt) {
    const LayerDev& L = p.L;
    const bool dec = (p.mode == kModeDecode);
    if (p.defer && tt == 0) {
        // A deferred launch orders only its end behind the previous kernel: this thread, idle
        // until the first unit completes, sits out that kernel's last microseconds and then
        // lets the next launch in.
        ptx::griddep_wait();
        ptx::griddep_launch_dependents();
        MKV_TR(7);
    }
    // Which units this CTA looks after: the unit it starts in, if it is the first CTA to start
    // there, and the units after it in which no CTA starts, if it is the last one to start there.
    // Those are the units it streams first, in this order, so they also complete in this order
    // (a launch over many layers has more units than CTAs).
    const int c = (int)blockIdx.x;
    const int u_first = L.cta_unit0[c];
    const bool first_there = (c == 0) || (L.cta_unit0[c - 1] != u_first);
    const bool last_there = (c + 1 == (int)gridDim.x) || (L.cta_unit0[c + 1] != u_first);
    const int u_begin = first_there ? u_first : u_first + 1;
    const int u_end = last_there ? ((c + 1 == (int)gridDim.x) ? L.n_units : L.cta_unit0[c + 1]) : u_first + 1;
    for (int u = u_begin; u < u_end; ++u) {
        TailPre<kTailThreads, GB> pre;
        tail_prefetch<__nv_bfloat16, kTailThreads, GB, LAYER>(p, u, *tsm, tt, pre);
        if (tt == 0) {
            const int total = p.det ? L.tile_begin[u + 1] - L.tile_begin[u]
                                    : unit_tiles(L.unit_lp[u], min(pre.n_dec, p.cap - (dec ? 1 : 0)));
            const unsigned long long t0 = ptx::globaltimer_ns();
            int slots = -1;
            int par = tsm->par;
            while (par < 0) {
                par = *reinterpret_cast<const volatile int*>(&ctl->par);
                if (par >= 0) { tsm->par = par; break; }
                if (aborted(ctl)) break;
                if (ptx::globaltimer_ns() - t0 > p.wait_ns) { note_timeout(p, ctl); break; }
            }
            const int2* cnt_u = L.cnt + (size_t)max(par, 0) * L.n_units + u;
            for (; par >= 0;) {
                const unsigned long long w = *reinterpret_cast<const volatile unsigned long long*>(cnt_u);
                if ((int)(unsigned)(w & 0xffffffffull) >= total) { slots = (int)(unsigned)(w >> 32); break; }
                if (aborted(ctl)) break;
                if (ptx::globaltimer_ns() - t0 > p.wait_ns) { note_timeout(p, ctl); break; }
                __nanosleep(100);
            }
            ctl->tail_unit = slots;
        }
        bar_sync(1, kTailThreads);
        const int slots = ctl->tail_unit;
        bar_sync(1, kTailThreads);
        if (slots < 0) break;
        __threadfence();
        if (tt == 0) MKV_TR_ADD(6, 1);
        if constexpr (LAYER) layer_unit_tail<__nv_bfloat16, kTailThreads, 1, GB>(p, u, slots, pre, *tsm, tt);
        else unit_tail<__nv_bfloat16, kTailThreads, 1, GB>(p, u, slots, pre, *tsm, tt);
        if (tt == 0) MKV_TR(5);
    }
}

template <bool LAYER>
__global__ void __launch_bounds__(kThreads, 2) mma_kernel(const Params p, const int nst) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* const stages = smem;
    uint8_t* const qslots = smem + (size_t)nst * kStageBytes;
    TailSmem<kTailThreads>* const tsm =
        reinterpret_cast<TailSmem<kTailThreads>*>(qslots + (size_t)kQSlots * kQSlotBytes);
    Control* const ctl = reinterpret_cast<Control*>(reinterpret_cast<uint8_t*>(tsm) + ((sizeof(TailSmem<kTailThreads>) + 15) & ~size_t(15)));

    const LayerDev& L = p.L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool dec = (p.mode == kModeDecode);
    const int G = p.group;

    if (tid == 0) {
        for (int s = 0; s < nst; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), kConsumerWarps);
            ptx::mbar_init(ptx::smem_u32(&ctl->xfull[s]), kConsumerWarps);
        }
        for (int s = 0; s < kQSlots; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctl->qfull[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl->qempty[s]), kConsumerWarps);
        }
        ctl->abort_flag = 0;
        ctl->tail_unit = -1;
        ctl->par = -1;
        tsm->par = -1;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    __syncthreads();
    if (tid == 0) { MKV_TR(0); MKV_TR_SET(6, 0); }
    const bool defer = p.defer != 0;
    // The next kernel of the stream may begin once every CTA of this one has said so
    // (griddepcontrol.launch_dependents) -- which a CTA does only after it has itself passed the
    // dependency wait: when the next kernel runs, everything before this one is complete.

    if (warp == kProducerWarp) {
        // ================================ producer =====================================
        // Lane 0 issues copies and pulls chunks; all lanes help when a new unit must be found.
        int stage = 0;
        uint32_t phase = 0;
        uint32_t issued = 0;       // bit s: a copy into stage s may still be in flight
        uint32_t issued_par = 0;   // parity its full barrier completes with
        bool ok = true;
        // K and V are read exactly once per step: let them leave L2 first, so that the
        // step's scratch (logits, partials) and the scores stay resident for the tails
        const unsigned long long stream_policy = ptx::l2_policy_evict_first();
        int qcount = 0;            // visits that had at least one tile (and therefore a query slot)
        auto acquire = [&]() -> bool {
            if (!wait_or_abort(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.wait_ns)) {
                if (!aborted(ctl)) note_timeout(p, ctl);
                return false;
            }
            issued &= ~(1u << stage);
            return true;
        };
        auto advance = [&]() { if (++stage == nst) { stage = 0; phase ^= 1u; } };
        auto issue_tile = [&](int u, const TileRef& tr, int first, int pre) -> bool {
            if (!acquire()) return false;
            StageMeta& mt = ctl->meta[stage];
            mt.kind = kEntryTile; mt.unit = u; mt.seg = tr.seg; mt.row = tr.row; mt.cnt = tr.cnt; mt.first = first;
            mt.pre = pre;
            const uint32_t fb = ptx::smem_u32(&ctl->full[stage]);
            const uint32_t dstK = ptx::smem_u32(stages + (size_t)stage * kStageBytes);
            const size_t off = ((size_t)u * (tr.seg == 0 ? p.max_prefill : p.cap) + tr.row) * kRowB;
            const uint8_t* kb = (tr.seg == 0 ? L.Kp : L.Kd) + off;
            const uint8_t* vb = (tr.seg == 0 ? L.Vp : L.Vd) + off;
            const uint32_t bytes = (uint32_t)tr.cnt * kRowB;
            ptx::mbar_arrive_expect_tx(fb, 2u * bytes);
            ptx::bulk_g2s_hint(dstK, kb, bytes, fb, stream_policy);
            ptx::bulk_g2s_hint(dstK + kTileBytes, vb, bytes, fb, stream_policy);
            issued |= 1u << stage;
            issued_par = (issued_par & ~(1u << stage)) | (phase << stage);
            advance();
            return true;
        };
        // the unit's G query rows, one padded row each, into the next query slot
        auto issue_query = [&](int u) -> bool {
            const int b = u / p.kv_heads, g = u - b * p.kv_heads;
            const int qi = qcount & 1;
            if (!wait_or_abort(ptx::smem_u32(&ctl->qempty[qi]), (uint32_t)(((qcount >> 1) & 1) ^ 1), ctl, p.wait_ns)) {
                if (!aborted(ctl)) note_timeout(p, ctl);
                return false;
            }
            const uint32_t qb = ptx::smem_u32(&ctl->qfull[qi]);
            const uint8_t* qsrc = reinterpret_cast<const uint8_t*>(p.q) + ((size_t)b * p.q_heads + (size_t)g * G) * kRowB;
            ptx::mbar_arrive_expect_tx(qb, (uint32_t)G * kRowB);
            for (int h = 0; h < G; ++h)
                ptx::bulk_g2s(ptx::smem_u32(qslots + (size_t)qi * kQSlotBytes + (size_t)h * kQRowB),
                              qsrc + (size_t)h * kRowB, kRowB, qb);
            ++qcount;
            if (dec) {   // the tail will want the fresh token's rows: bring them into L2 now
                const uint8_t* kn = reinterpret_cast<const uint8_t*>(p.k_new) + (size_t)u * kRowB;
                const uint8_t* vn = reinterpret_cast<const uint8_t*>(p.v_new) + (size_t)u * kRowB;
                ptx::prefetch_l2(kn); ptx::prefetch_l2(kn + 128);
                ptx::prefetch_l2(vn); ptx::prefetch_l2(vn + 128);
            }
            return true;
        };
        const int U = L.n_units;
        int u = L.cta_unit0[blockIdx.x];
        int lp = L.unit_lp[u];
        // state of the current unit visit (lane 0)
        int sent = 0;              // tile entries sent
        int mine = 0;              // tiles covered, empty ones included
        int slot = -1;             // the visit's partial slot (taken with the first tile)
        bool q_sent = false;
        // Before the dependency wait only data no earlier kernel of the stream writes may be
        // touched: the start table and the frozen prefill pool.  The CTA's reserved tiles (prefill
        // tiles by construction) are therefore in flight while the previous step still runs.
        int head_t = 0, head_end = 0;   // reserved tiles still to issue (lane 0)
        const bool early = p.early_inputs != 0;
        if (lane == 0) {
            head_t = L.cta_head0[blockIdx.x];
            head_end = head_t + L.cta_headn[blockIdx.x];
            // With early inputs the query is final already and the consumers work through the
            // reserved tiles now; otherwise no more than the ring holds, for the consumers only
            // start after the wait.
            if (early && head_t < head_end) { ok = issue_query(u); q_sent = true; }
            const int before = early ? head_end - head_t : nst;
            for (int n = 0; head_t < head_end && n < before && ok; ++n, ++head_t) {
                ok = issue_tile(u, tile_ref(head_t, lp, 0), sent == 0, early ? 1 : 0);
                if (ok) { if (sent == 0) MKV_TR(1); ++sent; ++mine; }
            }
        }
        if (!defer) {
            ptx::griddep_wait();
            ptx::griddep_launch_dependents();
        }
        if (lane == 0 && !defer) MKV_TR(7);
        // Loads first, then the query copy, then their use: the consumers wait for the query, which
        // must not wait for a load's round trip.
        int n_old = L.n_dec[u];
        uint32_t seen = 0;         // launches this CTA has taken part in (lane 0)
        if (lane == 0) seen = __ldcg(&L.launch_no[blockIdx.x]);
        const bool has_head = head_end > L.cta_head0[blockIdx.x];
        if (lane == 0 && ok && has_head && !q_sent) {
            ok = issue_query(u);
            q_sent = true;
        }
        n_old = min(n_old, p.cap - (dec ? 1 : 0));
        // which copy of the unit counters this launch uses
        int par = 0;
        if (lane == 0) {
            par = (int)(seen & 1u);
            L.launch_no[blockIdx.x] = seen + 1u;
            *reinterpret_cast<volatile int*>(&ctl->par) = par;
        }
        par = __shfl_sync(0xffffffffu, par, 0);
        int32_t* const nxt = L.next + (size_t)par * L.n_units;
        int2* const cnt = L.cnt + (size_t)par * L.n_units;
        int total = unit_tiles(lp, n_old);
        int chunk = L.unit_chunk[u];
        if (lane == 0 && ok && has_head) {
            slot = (int)(count_add(&cnt[u], 1ull << 32) >> 32);
            for (; head_t < head_end && ok; ++head_t) {
                ok = issue_tile(u, tile_ref(head_t, lp, 0), sent == 0, 0);
                ++sent; ++mine;
            }
        }
        // Reproducible mode: this CTA's fixed range of the global tile sequence, unit by unit; the
        // partial of a unit visit goes to the slot that is this CTA's rank among the unit's CTAs.
        if (p.det && lane == 0 && ok) {
            int t = L.cta_t0[blockIdx.x];
            const int t_end = L.cta_t0[blockIdx.x + 1];
            for (int uu = u; t < t_end && ok; ++uu) {
                const int ub = L.tile_begin[uu], ue = L.tile_begin[uu + 1];
                const int lpu = L.unit_lp[uu];
                const int ndu = min(L.n_dec[uu], p.cap - (dec ? 1 : 0));
                const int a = t - ub, b = min(t_end, ue) - ub;
                count_add(&cnt[uu], 1ull << 32);               // visits of the unit (the tail's partial count)
                int sent_u = 0;
                for (int tt = a; tt < b && ok; ++tt) {
                    const TileRef tr = tile_ref(tt, lpu, ndu);
                    if (tr.cnt == 0) continue;
                    if (sent_u == 0 && !(ok = issue_query(uu))) break;
                    ok = issue_tile(uu, tr, sent_u == 0, 0);
                    ++sent_u;
                }
                if (ok && (ok = acquire())) {
                    StageMeta& mt = ctl->meta[stage];
                    mt.kind = kEntryExchange; mt.unit = uu; mt.seg = 0; mt.row = 0; mt.cnt = 0; mt.first = (sent_u == 0);
                    mt.slot = (int)blockIdx.x - L.unit_cta0[uu]; mt.ntiles = b - a; mt.total = ue - ub; mt.pre = 0;
                    ptx::mbar_arrive(ptx::smem_u32(&ctl->full[stage]));
                    advance();
                }
                t = ub + b;
            }
        }
        int g = 0;                 // first tile of the chunk in hand
        if (lane == 0 && !p.det) g = atomicAdd(&nxt[u], chunk);
        for (; !p.det;) {
            g = __shfl_sync(0xffffffffu, g, 0);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            if (g < total) {
                if (lane == 0) {
                    const int g_next = atomicAdd(&nxt[u], chunk);   // in flight while this chunk is issued
                    if (slot < 0) slot = (int)(count_add(&cnt[u], 1ull << 32) >> 32);
                    const int t_end = min(g + chunk, total);
                    for (int t = g; t < t_end && ok; ++t) {
                        const TileRef tr = tile_ref(t, lp, n_old);
                        ++mine;
                        if (tr.cnt == 0) continue;
                        if (!q_sent) { ok = issue_query(u); q_sent = true; if (!ok) break; }
                        ok = issue_tile(u, tr, sent == 0, 0);
                        ++sent;
                    }
                    g = g_next;
                }
                continue;
            }
            // The unit has no tiles left to hand out: deliver this visit ...
            if (lane == 0 && mine > 0) {
                if ((ok = acquire())) {
                    StageMeta& mt = ctl->meta[stage];
                    mt.kind = kEntryExchange; mt.unit = u; mt.seg = 0; mt.row = 0; mt.cnt = 0; mt.first = (sent == 0);
                    mt.slot = slot; mt.ntiles = mine; mt.total = total; mt.pre = 0;
                    ptx::mbar_arrive(ptx::smem_u32(&ctl->full[stage]));
                    advance();
                }
                sent = 0; mine = 0; slot = -1; q_sent = false;
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            // ... and look for the next unit (cyclically after this one) that still has some.
            int found = -1;
            for (int base = 1; base < U && base <= kHopWindow && found < 0; base += 32) {
                const int k = base + lane;
                int lpc = 0, ndc = 0, rem = 0, chc = 2;
                if (k < U) {
                    const int cand = (u + k) % U;
                    lpc = L.unit_lp[cand];
                    chc = L.unit_chunk[cand];
                    ndc = min(L.n_dec[cand], p.cap - (dec ? 1 : 0));
                    rem = max(0, unit_tiles(lpc, ndc) - __ldcg(&nxt[cand]));
                }
                // of these 32 units take the one with the most tiles left (the nearest on a tie):
                // help goes where a slow CTA has fallen behind, and fewer visits end after one chunk
                int best = (rem << 5) | (31 - lane);
#pragma unroll
                for (int off = 16; off; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
                if (best >> 5) {
                    const int src = 31 - (best & 31);
                    found = (u + base + src) % U;
                    lp = __shfl_sync(0xffffffffu, lpc, src);
                    n_old = __shfl_sync(0xffffffffu, ndc, src);
                    chunk = __shfl_sync(0xffffffffu, chc, src);
                }
            }
            if (found < 0) break;
            u = found;
            total = unit_tiles(lp, n_old);
            if (lane == 0) g = atomicAdd(&nxt[u], chunk);
        }
        if (lane == 0) {
            if (ok && acquire()) {
                ctl->meta[stage].kind = kEntryEnd;
                ctl->meta[stage].pre = 0;
                ptx::mbar_arrive(ptx::smem_u32(&ctl->full[stage]));
            } else {
                // abort: leave only after every copy this thread issued has landed
                for (int s2 = 0; s2 < nst; ++s2)
                    if (issued & (1u << s2))
                        ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->full[s2]), (issued_par >> s2) & 1u, p.wait_ns);
            }
        }
        __syncwarp();
    } else if (warp < kConsumerWarps) {
        // ================================ consumers ====================================
        // They pass the dependency wait at the first entry that was issued after the producer's
        // own: entries issued before it (reserved prompt tiles, with early inputs) read frozen
        // rows and the caller's query only, and change nothing but registers.
        bool waited = false;
        int stage = 0;
        uint32_t phase = 0;
        int xcount = 0;
        float oacc[8][4];              // O^T: [16-dim block][dim 0-7 | 8-15 x head pair]
        float m_run = kNegBig, l_run = 0.f;
        int qcount = 0;
        const uint8_t* qs = qslots;    // this lane's place in the current query slot
        const int head = lane >> 2, tk0 = 2 * (lane & 3);
        const int mi = lane >> 3, rr = lane & 7;
        const int blk0 = warp * 16;
        float* lg = L.logit;           // this lane's head row of the unit's logit scratch
#pragma unroll
        for (int j = 0; j < 8; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }

        for (;;) {
            if (!wait_or_abort(ptx::smem_u32(&ctl->full[stage]), phase, ctl, p.wait_ns)) {
                if (lane == 0 && !aborted(ctl)) note_timeout(p, ctl);
                break;
            }
            const StageMeta mt = ctl->meta[stage];
            if (!waited && !mt.pre && !defer) { ptx::griddep_wait(); waited = true; }
            if (warp == 0 && lane == 0 && xcount == 0 && mt.first) MKV_TR(2);
            if (mt.kind == kEntryEnd) {
                if (warp == 0 && lane == 0) MKV_TR(3);
                const int xs = xcount % nst;           // tells the tail warps that nothing follows
                if (warp == 0 && lane == 0) ctl->xq[xs].stage = -1;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->xfull[xs]));
                break;
            }
            uint8_t* const sK = stages + (size_t)stage * kStageBytes;
            uint8_t* const sV = sK + kTileBytes;
            if (mt.first) {
                m_run = kNegBig; l_run = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }
                {
                    const int b = mt.unit / p.kv_heads, g = mt.unit - b * p.kv_heads;
                    lg = L.logit + ((size_t)b * p.q_heads + (size_t)g * G + min(head, G - 1)) * p.lstride;
                }
                if (mt.kind == kEntryTile) {
                    const int qi = qcount & 1;
                    if (!wait_or_abort(ptx::smem_u32(&ctl->qfull[qi]), (uint32_t)((qcount >> 1) & 1), ctl, p.wait_ns)) {
                        if (lane == 0 && !aborted(ctl)) note_timeout(p, ctl);
                        break;
                    }
                    qs = qslots + (size_t)qi * kQSlotBytes + (size_t)head * kQRowB + tk0 * 2;
                }
            }
            if (mt.kind == kEntryTile) {
                const int nv = mt.cnt;
                bool wrote = false;
                if (nv > blk0 && nv < blk0 + 16) {
                    // rows past the valid ones enter the second mma with probability 0: their V
                    // bytes must be finite, so clear them (stale shared memory may hold anything)
                    const int nz = (blk0 + 16 - nv) * 16;
                    for (int idx = lane; idx < nz; idx += 32)
                        *reinterpret_cast<uint4*>(sV + (size_t)(nv + (idx >> 4)) * kRowB + ((idx & 15) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    wrote = true;
                    __syncwarp();
                }
                if (nv > blk0) {
                    // ---------------- S = Q K^T: 8 heads (M, padded to 16) x 16 tokens -------------
                    float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                    const uint32_t roff = (uint32_t)(blk0 + (mi >> 1) * 8 + rr) * kRowB;
                    const uint32_t kbase = ptx::smem_u32(sK) + roff;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        uint32_t b00, b01, b10, b11;
                        ptx::ldmatrix_x4(kbase + (uint32_t)(((2 * ks + (mi & 1)) ^ rr) << 4), b00, b01, b10, b11);
                        // A fragment: this head's query elements (rows past G are zero)
                        uint32_t qa0 = *reinterpret_cast<const uint32_t*>(qs + 32 * ks);
                        uint32_t qa1 = *reinterpret_cast<const uint32_t*>(qs + 32 * ks + 16);
                        if (head >= G) { qa0 = 0u; qa1 = 0u; }
                        ptx::mma_bf16(sacc[0], qa0, 0u, qa1, 0u, b00, b01);
                        ptx::mma_bf16(sacc[1], qa0, 0u, qa1, 0u, b10, b11);
                    }
                    // ---------------- online softmax in registers (fp32) -------------------------
                    float s[4] = {sacc[0][0], sacc[0][1], sacc[1][0], sacc[1][1]};
                    const int trow[4] = {blk0 + tk0, blk0 + tk0 + 1, blk0 + tk0 + 8, blk0 + tk0 + 9};
#pragma unroll
                    for (int i = 0; i < 4; ++i) s[i] = (trow[i] < nv) ? s[i] * p.scale_log2 : kNegBig;
                    if (dec && mt.seg == 1 && head < G) {
                        float* lr = lg + mt.row;
                        if (trow[1] < nv) *reinterpret_cast<float2*>(lr + trow[0]) = make_float2(s[0], s[1]);
                        else if (trow[0] < nv) lr[trow[0]] = s[0];
                        if (trow[3] < nv) *reinterpret_cast<float2*>(lr + trow[2]) = make_float2(s[2], s[3]);
                        else if (trow[2] < nv) lr[trow[2]] = s[2];
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
                    if (__any_sync(0xffffffffu, sc != 1.0f)) {
                        // O^T holds heads 2*(lane&3) and +1 in its columns: fetch their factors
                        const float scA = __shfl_sync(0xffffffffu, sc, (lane & 3) * 8);
                        const float scB = __shfl_sync(0xffffffffu, sc, (lane & 3) * 8 + 4);
#pragma unroll
                        for (int j = 0; j < 8; ++j) { oacc[j][0] *= scA; oacc[j][1] *= scB; oacc[j][2] *= scA; oacc[j][3] *= scB; }
                    }
                    // P^T as B operand (tokens in K, heads in N).  P = hi + lo in bf16: the
                    // product with V then carries ~16 mantissa bits of P.
                    const uint32_t bhi0 = ptx::pack_bf16x2(pr[0], pr[1]);
                    const uint32_t bhi1 = ptx::pack_bf16x2(pr[2], pr[3]);
                    const uint32_t blo0 = ptx::pack_bf16x2(pr[0] - __uint_as_float(bhi0 << 16),
                                                           pr[1] - __uint_as_float(bhi0 & 0xffff0000u));
                    const uint32_t blo1 = ptx::pack_bf16x2(pr[2] - __uint_as_float(bhi1 << 16),
                                                           pr[3] - __uint_as_float(bhi1 & 0xffff0000u));
                    // ---------------- O^T += V^T P^T -------------------------------------------------
                    const uint32_t vbase = ptx::smem_u32(sV) + roff;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t a0, a1, a2, a3;
                        ptx::ldmatrix_x4_trans(vbase + (uint32_t)(((2 * j + (mi & 1)) ^ rr) << 4), a0, a1, a2, a3);
                        ptx::mma_bf16(oacc[j], a0, a1, a2, a3, bhi0, bhi1);
                        ptx::mma_bf16(oacc[j], a0, a1, a2, a3, blo0, blo1);
                    }
                }
                if (wrote) ptx::fence_proxy_async();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->empty[stage]));
            } else {
                // ---------------- item end: hand (m, l, O) to the tail warps ------------------------
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
                float* xo = reinterpret_cast<float*>(sK);
                float* xm = xo + kConsumerWarps * kMaxGroup * kXoStride;
                float* xl = xm + kConsumerWarps * kMaxGroup;
                if ((lane & 3) == 0) { xm[warp * kMaxGroup + head] = m_run; xl[warp * kMaxGroup + head] = l_run; }
                float* oA = xo + (size_t)(warp * kMaxGroup + tk0) * kXoStride + head;   // head tk0, dim lane>>2
                float* oB = oA + kXoStride;                                              // head tk0 + 1
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    oA[16 * j] = oacc[j][0]; oB[16 * j] = oacc[j][1];
                    oA[16 * j + 8] = oacc[j][2]; oB[16 * j + 8] = oacc[j][3];
                }
                if (!mt.first) {     // the item had tiles: its query slot is free again
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->qempty[qcount & 1]));
                    ++qcount;
                }
                const int xs = xcount % nst;
                if (warp == 0 && lane == 0) { ctl->xq[xs].stage = stage; ctl->xq[xs].unit = mt.unit; ctl->xq[xs].slot = mt.slot;
                                             ctl->xq[xs].ntiles = mt.ntiles; ctl->xq[xs].total = mt.total; }
                ptx::fence_proxy_async();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->xfull[xs]));
                ++xcount;
            }
            if (++stage == nst) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == kMergeWarp) {
        // ================================ merge warp ===================================
        // Folds the four consumer states of a unit visit into one partial in global memory,
        // gives the borrowed stage back, adds the visit's tiles to the unit's count and, when
        // that completes the unit, publishes the unit in the layer's queue of due tails.
        if (!defer) ptx::griddep_wait();
        for (int x = 0;; ++x) {
            const int xs = x % nst;
            if (!wait_or_abort(ptx::smem_u32(&ctl->xfull[xs]), (uint32_t)((x / nst) & 1), ctl, p.wait_ns)) {
                if (lane == 0 && !aborted(ctl)) note_timeout(p, ctl);
                break;
            }
            const ExchangeRef ref = ctl->xq[xs];
            if (ref.stage < 0) break;
            const int u = ref.unit;
            if (ref.slot < 0 || ref.slot >= kMaxParts) {     // cannot happen: chunks are sized to prevent it
                if (lane == 0) atomicCAS(p.status, kStatusOk, kStatusDeviceCheck);
            }
            const float* xo = reinterpret_cast<const float*>(stages + (size_t)ref.stage * kStageBytes);
            const float* xm = xo + kConsumerWarps * kMaxGroup * kXoStride;
            const float* xl = xm + kConsumerWarps * kMaxGroup;
            const size_t part = (size_t)u * kMaxParts + (size_t)min(max(ref.slot, 0), kMaxParts - 1);
            for (int h = 0; h < G; ++h) {
                float M = xm[h];
#pragma unroll
                for (int w = 1; w < kConsumerWarps; ++w) M = fmaxf(M, xm[w * kMaxGroup + h]);
                float wsc[kConsumerWarps];
                float ls = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    wsc[w] = fast_exp2(xm[w * kMaxGroup + h] - M);
                    ls = fmaf(xl[w * kMaxGroup + h], wsc[w], ls);
                }
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float4 v = *reinterpret_cast<const float4*>(xo + (size_t)(w * kMaxGroup + h) * kXoStride + 4 * lane);
                    acc.x = fmaf(v.x, wsc[w], acc.x); acc.y = fmaf(v.y, wsc[w], acc.y);
                    acc.z = fmaf(v.z, wsc[w], acc.z); acc.w = fmaf(v.w, wsc[w], acc.w);
                }
                *reinterpret_cast<float4*>(&L.part_o[(part * G + h) * 128 + 4 * lane]) = acc;
                if (lane == 0) *reinterpret_cast<float2*>(&L.part_ml[(part * G + h) * 2]) = make_float2(M, ls);
            }
            __syncwarp();
            ptx::fence_proxy_async();
            // the borrowed stage goes back to the producer (its empty barrier counts four arrivals)
            if (lane < kConsumerWarps) ptx::mbar_arrive(ptx::smem_u32(&ctl->empty[ref.stage]));
            __threadfence();
            __syncwarp();
            if (lane == 0) {
                MKV_TR(4);
                // (the producer wrote the parity before it sent this visit's first counter pull)
                const int par = *reinterpret_cast<const volatile int*>(&ctl->par);
                count_add(&L.cnt[(size_t)par * L.n_units + u], (unsigned long long)ref.ntiles);
            }
        }
    } else {
        // ================================ tail warps ===================================
        if (!defer) ptx::griddep_wait();
        if (G <= 4) tail_group<4, LAYER>(p, ctl, tsm, tid - kTailTid0);
        else tail_group<8, LAYER>(p, ctl, tsm, tid - kTailTid0);
    }
}

}  // namespace

#ifdef MKV_TRACE
extern "C" __attribute__((visibility("default"))) int mkv_debug_trace(unsigned long long* host, int n) {
    return (int)cudaMemcpyFromSymbol(host, g_trace, sizeof(unsigned long long) * n);
}
#endif

bool mma_supported(int kv_dtype, int head_dim, int group) {
    return kv_dtype == 0 && head_dim == 128 && group >= 1 && group <= kMaxGroup;
}

int mma_max_stages() {
    int n = 2;
    while (n < kMaxStages && smem_bytes(n + 1) <= kSmemPerCta) ++n;
    return n;
}

// CTAs of the kernel an SM keeps resident with a ring of `stages` stages.  Also raises the
// kernels' dynamic shared memory limit to what that ring needs.
cudaError_t mma_occupancy(int stages, int* resident_per_sm) {
    static size_t opted = 0;       // the limit is a per-function maximum: it only ever grows
    const size_t need = smem_bytes(stages);
    if (need > kSmemPerCta) return cudaErrorInvalidValue;
    if (need > opted) {
        cudaError_t e = cudaFuncSetAttribute(mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
        if (e != cudaSuccess) return e;
        opted = need;
    }
    int a = 0, b = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, mma_kernel<false>, kThreads, need);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, mma_kernel<true>, kThreads, need);
    if (e != cudaSuccess) return e;
    *resident_per_sm = a < b ? a : b;
    return cudaSuccess;
}

// overlap: launch with programmatic stream serialization, i.e. this kernel's CTAs may start
// while the previous kernel of the stream is still finishing; the kernel itself waits
// (griddepcontrol.wait) before it touches anything an earlier kernel may write.
cudaError_t launch_mma(const Params& p, cudaStream_t st, bool overlap, int stages) {
    if (p.L.n_ctas <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.L.n_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes(stages);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    // the layer-wide score mode has its own instantiation, so that neither carries the other's tail
    if (p.layer_mean) return cudaLaunchKernelEx(&cfg, mma_kernel<true>, p, stages);
    return cudaLaunchKernelEx(&cfg, mma_kernel<false>, p, stages);
}

}  // namespace mkv
