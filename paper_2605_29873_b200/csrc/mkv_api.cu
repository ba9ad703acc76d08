// C ABI of the Moment-KV decode library: argument checks, workspace carving, the CTAs'
// start table, launches.  All device work is in the kernels; nothing here computes any
// step of the method on the host.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/mkv.h"
#include "mkv_launch.h"
#include "mkv_ptx.cuh"

using namespace mkv;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int round4(int a) { return (a + 3) / 4 * 4; }
inline int elem_size(int dt) { return dt == MKV_BF16 ? 2 : 4; }

// State arrays are stored for all layers back to back: `off` is layer 0's part, `stride` the
// bytes of one layer, with no padding in between, so that layers [l0, l0 + n) are one array of
// n * units units.
struct ArrOff { size_t off, stride; };
struct StateOff {
    ArrOff Kp, Vp, Kd, Vd, score, pos, n_dec, abar, abar_pos, n_prev, ev_k, ev_pos, ev_score, unit_lp, unit_step,
        seq_ticket;
};
// Scratch that lives for one step only, shared by all launches of the context (calls on a
// context are ordered on one stream, and a step touches it only after every earlier kernel
// of the stream has completed).  Sized for a launch over all layers.  It exists twice and
// launches alternate between the two sets, so that a launch which does not wait for its
// predecessor (see Params::defer) never shares scratch with it.
struct ScratchOff { size_t logit, head_sum, unit_sum, part_o, part_ml, keys, list_a, list_b, end; };
// A launch plan: the CTAs' start table and the work-sharing counters of the launches that use it.
// There is one per layer (launches of that layer alone) and one more for launches over several
// layers, sized for all of them.
struct PlanOff {
    size_t cta_unit0, cta_head0, cta_headn, cta_t0, unit_next0, unit_chunk, tile_begin, unit_cta0, next, cnt,
        launch_no, end;
};
struct Layout {
    int layers, units, cap, rowb, lstride;
    size_t status, stage_q, stage_k, stage_v, stage_out, scratch0, scratch_bytes, state0, plans0, plan_bytes, total;
    ScratchOff so;  // offsets relative to the scratch base
    StateOff st;    // offsets relative to the state base
    PlanOff po;     // a single layer's plan, offsets relative to the plan's base
    PlanOff pso;    // the several-layer plan, relative to its base (after the per-layer plans)
};

PlanOff make_plan_off(size_t nu) {
    PlanOff p;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    p.cta_unit0 = take((size_t)kMaxCtas * 4);
    p.cta_head0 = take((size_t)kMaxCtas * 4);
    p.cta_headn = take((size_t)kMaxCtas * 4);
    p.cta_t0 = take((size_t)(kMaxCtas + 1) * 4);
    p.unit_next0 = take(nu * 4);
    p.unit_chunk = take(nu * 4);
    p.tile_begin = take((nu + 1) * 4);
    p.unit_cta0 = take(nu * 4);
    p.next = take(2 * nu * 4);      // two copies each, alternating from launch to launch
    p.cnt = take(2 * nu * 8);
    p.launch_no = take((size_t)kMaxCtas * 4);   // per CTA: launches since the plan was (re)built
    p.end = o;
    return p;
}

bool make_layout(int layers, int batch, int q_heads, int kv_heads, int head_dim, int budget, int max_prefill,
                 int kv_dtype, Layout* out) {
    if (layers < 1 || batch < 1 || q_heads < 1 || kv_heads < 1 || budget < 1 || max_prefill < 0) return false;
    if (q_heads % kv_heads) return false;
    if (head_dim != 64 && head_dim != 128) return false;
    if (kv_dtype != MKV_BF16 && kv_dtype != MKV_F32) return false;
    const int G = q_heads / kv_heads;
    if (G > kMaxGroup) return false;
    if ((long long)budget + 1 > (1 << 24) || max_prefill > (1 << 24)) return false;
    if ((long long)layers * batch * kv_heads > (1 << 24)) return false;
    Layout L;
    L.layers = layers;
    L.units = batch * kv_heads;
    L.cap = budget + 1;
    L.rowb = head_dim * elem_size(kv_dtype);
    L.lstride = round4(L.cap);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    L.status = take(256);
    L.stage_q = take((size_t)batch * q_heads * head_dim * 4);
    L.stage_k = take((size_t)batch * kv_heads * head_dim * 4);
    L.stage_v = take((size_t)batch * kv_heads * head_dim * 4);
    L.stage_out = take((size_t)batch * q_heads * head_dim * 4);
    L.scratch0 = o;
    const size_t U = (size_t)L.units, C = (size_t)L.cap, NL = (size_t)layers, UA = U * NL;
    o = 0;
    L.so.logit = take(NL * batch * q_heads * L.lstride * 4);
    L.so.head_sum = take(NL * batch * L.lstride * 4);   // zero from mkv_create's memset, kept zero by its users
    L.so.unit_sum = take(UA * L.lstride * 4);
    L.so.part_o = take(UA * kMaxParts * G * head_dim * 4);
    L.so.part_ml = take(UA * kMaxParts * G * 2 * 4);
    L.so.keys = take(UA * C * 8);
    L.so.list_a = take(UA * C * 4);
    L.so.list_b = take(UA * C * 4);
    L.so.end = o;
    L.scratch_bytes = o;
    L.state0 = L.scratch0 + 2 * o;
    o = 0;
    auto arr = [&](size_t bytes_per_layer) { ArrOff a{o, bytes_per_layer}; o = align_up(o + bytes_per_layer * NL); return a; };
    L.st.Kp = arr(U * max_prefill * L.rowb);
    L.st.Vp = arr(U * max_prefill * L.rowb);
    L.st.Kd = arr(U * C * L.rowb);
    L.st.Vd = arr(U * C * L.rowb);
    L.st.score = arr(U * L.lstride * 4);
    L.st.pos = arr(U * L.lstride * 4);
    L.st.n_dec = arr(U * 4);
    L.st.abar = arr(U * C * 4);
    L.st.abar_pos = arr(U * C * 4);
    L.st.n_prev = arr(U * 4);
    L.st.ev_k = arr(U * 4);
    L.st.ev_pos = arr(U * C * 4);
    L.st.ev_score = arr(U * C * 4);
    L.st.unit_lp = arr(U * 4);
    L.st.unit_step = arr(U * 4);
    L.st.seq_ticket = arr((size_t)batch * 4);
    L.plans0 = L.state0 + o;
    L.po = make_plan_off(U);
    L.pso = make_plan_off(UA);
    L.plan_bytes = L.po.end;
    L.total = L.plans0 + L.plan_bytes * NL + L.pso.end;
    *out = L;
    return true;
}

// Copies source rows [units][src_rows][rowb] into the chunk-permuted pool rows.
__global__ void prefill_copy_kernel(const uint8_t* __restrict__ srcK, const uint8_t* __restrict__ srcV,
                                    uint8_t* __restrict__ dstK, uint8_t* __restrict__ dstV,
                                    const int32_t* __restrict__ unit_lp, int units, int src_rows, int max_prefill,
                                    int rowb) {
    const int chunks = rowb >> 4;
    const long long per_unit = (long long)src_rows * chunks;
    const long long total = per_unit * units;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int u = (int)(i / per_unit);
        const long long r = i - (long long)u * per_unit;
        const int row = (int)(r / chunks), c = (int)(r - (long long)row * chunks);
        if (row >= unit_lp[u]) continue;
        const size_t s = ((size_t)u * src_rows + row) * rowb + (size_t)c * 16;
        const size_t d = ((size_t)u * max_prefill + row) * rowb + (size_t)((c ^ (row & 7)) * 16);
        *reinterpret_cast<uint4*>(dstK + d) = *reinterpret_cast<const uint4*>(srcK + s);
        *reinterpret_cast<uint4*>(dstV + d) = *reinterpret_cast<const uint4*>(srcV + s);
    }
}

// The step's inputs from pinned host memory into the staging area, read over the bus by the
// GPU itself (16 bytes per thread).  Cheaper to start than a copy operation, and the step's
// kernel, launched right behind with programmatic serialization, may begin its own start-up
// meanwhile: it waits for this grid before it reads the staging area.
struct HostPiece { const uint4* src; uint4* dst; int n16; };
__global__ void host_gather_kernel(const HostPiece a, const HostPiece b, const HostPiece c3) {
    ptx::griddep_launch_dependents();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < a.n16) { a.dst[i] = a.src[i]; return; }
    i -= a.n16;
    if (i < b.n16) { b.dst[i] = b.src[i]; return; }
    i -= b.n16;
    if (i < c3.n16) c3.dst[i] = c3.src[i];
}

// Test hook of mkv_debug_inject: one tile of unit `u` counts as never delivered (both copies of
// its count start at -1), so its tail never becomes due.
__global__ void debug_kernel(LayerDev L, int u) {
    L.cnt[u] = make_int2(-1, 0);
    L.cnt[L.n_units + u] = make_int2(-1, 0);
}

// The device's view of pinned host memory [p, p + bytes), or nullptr if the GPU cannot read it
// in place (pageable memory, unknown pointer, not 16-byte aligned).
void* pinned_view(const void* p, size_t bytes) {
    cudaPointerAttributes a0, a1;
    if (cudaPointerGetAttributes(&a0, p) != cudaSuccess ||
        cudaPointerGetAttributes(&a1, (const uint8_t*)p + bytes - 1) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (a0.type != cudaMemoryTypeHost || a1.type != cudaMemoryTypeHost || !a0.devicePointer || !a1.devicePointer) return nullptr;
    if ((const uint8_t*)a1.devicePointer - (const uint8_t*)a0.devicePointer != (ptrdiff_t)(bytes - 1)) return nullptr;
    return ((uintptr_t)a0.devicePointer & 15u) == 0 ? a0.devicePointer : nullptr;
}

constexpr int kMinChunk = 2;   // tiles per pull of a unit's counter, lower bound

struct StartTable {
    int n_ctas = 0;
    std::vector<int32_t> lp, next0, chunk, cta_unit0, cta_head0, cta_headn;
    // reproducible mode
    std::vector<int32_t> tile_begin, cta_t0, unit_cta0;
};

// Start table.  A unit's rows are a sequence of 64-row tiles (prefill tiles, then decode
// tiles); the CTAs are spread over the units in proportion to the units' tile counts (a
// full decode pool assumed).  Each CTA owns `head_tiles` tiles outright at its place, if the
// unit has that many prefill tiles left to give (these can be fetched before the previous
// step has finished); everything else is handed out by the unit's counter, which
// therefore starts behind the reserved tiles.
//
// Every visit of a unit by a CTA that covers at least one tile delivers one partial, and a unit
// has room for kMaxParts of them.  Visits are bounded by the CTAs that start in the unit plus
// the successful pulls of its counter, so the table keeps the first below kMaxHome (the grid
// shrinks when few, long units would draw more) and sizes the unit's chunk -- tiles per pull --
// so that the second stays below kMaxParts - 8 - (CTAs starting there).
//
// det (reproducible mode): no counters.  The global tile sequence is cut into n_ctas contiguous
// ranges; CTA c covers tiles [cta_t0[c], cta_t0[c+1]) and delivers, for every unit its range
// reaches into, the partial number c - unit_cta0[unit].  Nothing is reserved.
StartTable build_start_table(int units, int budget, const int32_t* unit_lens, int n_ctas_max, int head_tiles,
                             bool det) {
    StartTable T;
    const int U = units;
    const int td = ceil_div(budget, kTileRows);
    T.lp.assign(U, 0);
    T.next0.assign(U, 0);
    std::vector<long long> tile_begin(U + 1, 0);
    for (int u = 0; u < U; ++u) {
        T.lp[u] = unit_lens[u];
        tile_begin[u + 1] = tile_begin[u] + ceil_div(T.lp[u], kTileRows) + td;
    }
    const long long t_all = tile_begin[U];
    long long t_max = 1;
    for (int u = 0; u < U; ++u) t_max = std::max(t_max, tile_begin[u + 1] - tile_begin[u]);
    // a unit of t tiles draws at most ceil(n_ctas * t / t_all) CTAs: keep that within kMaxHome
    const long long home_cap = (long long)(kMaxHome - 1) * t_all / t_max;
    int n_ctas = (int)std::max<long long>(1, std::min<long long>(std::min<long long>(n_ctas_max, t_all / 2), home_cap));
    // Units of equal size (a batch of equal prompts): make CTA stretches and units line up -- a
    // whole number of CTAs per unit, or a whole number of units per CTA -- so that no unit is
    // shared by CTAs that also serve its neighbours and most units end up with a single partial.
    bool equal = U > 1;
    for (int u2 = 1; u2 < U && equal; ++u2) equal = (tile_begin[u2 + 1] - tile_begin[u2]) == tile_begin[1];
    if (equal && !det) {
        if (n_ctas >= U) n_ctas = n_ctas / U * U;
        else n_ctas = ceil_div(U, ceil_div(U, n_ctas));
    }
    T.n_ctas = n_ctas;
    T.cta_unit0.assign(n_ctas, 0);
    T.cta_head0.assign(n_ctas, 0);
    T.cta_headn.assign(n_ctas, 0);
    T.cta_t0.assign(n_ctas + 1, 0);
    int u = 0;
    for (int cta = 0; cta < n_ctas; ++cta) {
        const long long t0 = t_all * cta / n_ctas;
        T.cta_t0[cta] = (int32_t)t0;
        while (tile_begin[u + 1] <= t0) ++u;
        T.cta_unit0[cta] = u;
        if (!det && head_tiles > 0 && T.next0[u] + head_tiles <= ceil_div(T.lp[u], kTileRows)) {
            T.cta_head0[cta] = T.next0[u];
            T.cta_headn[cta] = head_tiles;
            T.next0[u] += head_tiles;
        }
    }
    T.cta_t0[n_ctas] = (int32_t)t_all;
    std::vector<int> home(U, 0);
    for (int cta = 0; cta < n_ctas; ++cta) home[T.cta_unit0[cta]] += 1;
    T.chunk.assign(U, kMinChunk);
    for (int u2 = 0; u2 < U; ++u2) {
        const int pulls = kMaxParts - 8 - std::min(home[u2], kMaxHome);     // >= 24
        const int t = (int)(tile_begin[u2 + 1] - tile_begin[u2]) - T.next0[u2]; // tiles the counter hands out
        T.chunk[u2] = std::max(kMinChunk, ceil_div(std::max(t, 1), pulls));
    }
    T.tile_begin.assign(U + 1, 0);
    for (int u2 = 0; u2 <= U; ++u2) T.tile_begin[u2] = (int32_t)tile_begin[u2];
    // first CTA whose range [cta_t0[c], cta_t0[c+1]) reaches into the unit
    T.unit_cta0.assign(U, 0);
    int c = 0;
    for (int u2 = 0; u2 < U; ++u2) {
        while (c + 1 < n_ctas && T.cta_t0[c + 1] <= tile_begin[u2]) ++c;
        T.unit_cta0[u2] = c;
    }
    return T;
}

struct PinEntry { const void* host; size_t bytes; void* dev; };

}  // namespace

struct mkv_ctx {
    int layers, batch, q_heads, kv_heads, head_dim, group;
    int budget, budget_max, max_prefill;
    float beta;
    int kv_dtype, out_dtype, score_mode, kernel;
    unsigned flags;
    int device, sm_count;
    uint8_t* ws;
    Layout lay;
    int n_ctas_max; // persistent grid upper bound (SM count x CTAs that can be resident per SM)
    bool use_mma;
    int stages;     // ring depth of the tensor-core kernel
    int head_tiles; // tiles a CTA owns outright at its starting place
    int grid_share; // percent of n_ctas_max that a single-layer launch uses
    bool pdl;       // consecutive launches overlap (programmatic dependent launch)
    unsigned long long wait_ns;
    std::vector<char> prefilled;
    // per plan (layers single-layer plans, then the several-layer plan)
    std::vector<char> stepped;   // a launch has used the plan since it was (re)built
    std::vector<int> n_ctas;
    int stack_layer0, stack_n;   // layers the several-layer plan is built for (stack_n = 0: none)
    // the previous kernel launch of the context: its layers, stream and set of scratch
    int last_layer0, last_n, scratch_set;
    void* last_stream;
    std::vector<std::vector<int32_t>> lens;   // per layer, per (sequence, KV head) unit
    int64_t launches;
    std::vector<PinEntry> pins;  // host buffers already looked up by mkv_decode_step_host
};

namespace {

inline uint8_t* plan_base(const mkv_ctx* c, int plan) {
    return c->ws + c->lay.plans0 + c->lay.plan_bytes * (size_t)std::min(plan, c->layers);
}
inline const PlanOff& plan_off(const mkv_ctx* c, int plan) { return plan < c->layers ? c->lay.po : c->lay.pso; }

// Device view of layers [layer0, layer0 + n) as one list of n * units units, with launch plan `plan`.
LayerDev layer_dev(const mkv_ctx* c, int layer0, int n, int plan, int set = 0) {
    uint8_t* sb = c->ws + c->lay.scratch0 + c->lay.scratch_bytes * (size_t)set;
    uint8_t* stb = c->ws + c->lay.state0;
    uint8_t* pb = plan_base(c, plan);
    const StateOff& o = c->lay.st;
    const ScratchOff& so = c->lay.so;
    const PlanOff& po = plan_off(c, plan);
    auto at = [&](const ArrOff& a) { return stb + a.off + a.stride * (size_t)layer0; };
    LayerDev d;
    d.Kp = at(o.Kp); d.Vp = at(o.Vp); d.Kd = at(o.Kd); d.Vd = at(o.Vd);
    d.score = (float*)at(o.score);
    d.pos = (int32_t*)at(o.pos);
    d.n_dec = (int32_t*)at(o.n_dec);
    d.logit = (float*)(sb + so.logit);
    d.head_sum = (float*)(sb + so.head_sum);
    d.unit_sum = (float*)(sb + so.unit_sum);
    d.abar = (c->flags & MKV_FLAG_RECORD_PROBS) ? (float*)at(o.abar) : nullptr;
    d.abar_pos = (int32_t*)at(o.abar_pos);
    d.n_prev = (int32_t*)at(o.n_prev);
    d.ev_k = (int32_t*)at(o.ev_k);
    d.ev_pos = (int32_t*)at(o.ev_pos);
    d.ev_score = (float*)at(o.ev_score);
    d.n_units = c->lay.units * n;
    d.n_ctas = c->n_ctas[plan];
    d.cta_unit0 = (const int32_t*)(pb + po.cta_unit0);
    d.cta_head0 = (const int32_t*)(pb + po.cta_head0);
    d.cta_headn = (const int32_t*)(pb + po.cta_headn);
    d.cta_t0 = (const int32_t*)(pb + po.cta_t0);
    d.unit_lp = (const int32_t*)at(o.unit_lp);
    d.unit_next0 = (const int32_t*)(pb + po.unit_next0);
    d.unit_chunk = (const int32_t*)(pb + po.unit_chunk);
    d.tile_begin = (const int32_t*)(pb + po.tile_begin);
    d.unit_cta0 = (const int32_t*)(pb + po.unit_cta0);
    d.next = (int32_t*)(pb + po.next);
    d.cnt = (int2*)(pb + po.cnt);
    d.launch_no = (uint32_t*)(pb + po.launch_no);
    d.part_o = (float*)(sb + so.part_o);
    d.part_ml = (float*)(sb + so.part_ml);
    d.unit_step = (int32_t*)at(o.unit_step);
    d.seq_ticket = (int32_t*)at(o.seq_ticket);
    d.keys = (unsigned long long*)(sb + so.keys);
    d.list_a = (int32_t*)(sb + so.list_a);
    d.list_b = (int32_t*)(sb + so.list_b);
    return d;
}
LayerDev layer_dev(const mkv_ctx* c, int layer) { return layer_dev(c, layer, 1, layer); }

Params make_params(const mkv_ctx* c, int layer0, int n, int plan, const void* q, const void* k_new,
                   const void* v_new, void* out, int mode) {
    Params p;
    p.L = layer_dev(c, layer0, n, plan, c->scratch_set ^ 1);   // the set the previous launch did not use
    p.defer = 0;
    p.q = q; p.k_new = k_new; p.v_new = v_new; p.out = out;
    p.status = (int32_t*)(c->ws + c->lay.status);
    p.batch = c->batch * n; p.q_heads = c->q_heads; p.kv_heads = c->kv_heads; p.group = c->group;
    p.head_dim = c->head_dim;
    p.cap = c->lay.cap; p.max_prefill = c->max_prefill; p.budget = c->budget;
    p.lstride = c->lay.lstride;
    p.beta = c->beta;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)c->head_dim));
    p.mode = mode;
    // Eq. 4 over all heads of the layer: the tails of a sequence's KV heads work together
    p.layer_mean = (mode == kModeDecode && c->score_mode == MKV_SCORE_LAYER_MEAN && c->kv_heads > 1) ? 1 : 0;
    p.out_f32 = (c->out_dtype == MKV_F32);
    p.launch_parity = (int)(c->launches & 1);
    p.early_inputs = (c->flags & MKV_FLAG_INPUTS_READY) ? 1 : 0;
    p.det = (c->flags & MKV_FLAG_REPRODUCIBLE) ? 1 : 0;
    p.wait_ns = c->wait_ns;
    return p;
}

mkv_status launch_step(mkv_ctx* c, int plan, int layer0, int n, Params p, cudaStream_t st, bool staged_inputs = false) {
    // The first launch after a plan was (re)built must see the prefill's copies complete before
    // it reads the table and the pool; later ones may overlap their start with the previous
    // kernel's end.
    const bool overlap = c->pdl && c->stepped[plan];
    // A launch whose layers are all different from those of the context's previous launch on the
    // same stream has nothing in common with it (its own pools, scores and counters; the other
    // set of scratch), and with the caller's inputs final it need not wait for it at all.
    const bool disjoint = c->last_n > 0 && (layer0 >= c->last_layer0 + c->last_n || c->last_layer0 >= layer0 + n);
    p.defer = (overlap && c->use_mma && p.early_inputs && !staged_inputs && disjoint && c->last_stream == (void*)st) ? 1 : 0;
    cudaError_t e = c->use_mma ? launch_mma(p, st, overlap, c->stages) : launch_simt(p, c->kv_dtype, st);
    if (e != cudaSuccess) return MKV_ERR_CUDA;
    c->launches += 1;
    c->stepped[plan] = 1;
    c->last_layer0 = layer0; c->last_n = n; c->last_stream = (void*)st;
    c->scratch_set ^= 1;
    return MKV_OK;
}

bool layer_ok(const mkv_ctx* c, int layer) { return c && layer >= 0 && layer < c->layers; }
bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

struct DeviceGuard {
    int prev = -1; bool ok;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess;
        if (ok && prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Grid bound of the context's kernel family from what the device can keep resident.
mkv_status size_grid(mkv_ctx* c) {
    int resident = 0;
    const cudaError_t e = c->use_mma ? mma_occupancy(c->stages, &resident)
                                     : simt_occupancy(c->kv_dtype, c->head_dim, c->group, &resident);
    if (e != cudaSuccess) return MKV_ERR_CUDA;
    const int n = mkv_grid_limit(c->sm_count, resident, c->use_mma ? 2 : 8);
    if (n <= 0) return MKV_ERR_UNSUPPORTED;
    c->n_ctas_max = n;
    return MKV_OK;
}

// Writes a plan (start table, fresh counters) for `units` units with the given prompt lengths.
mkv_status upload_plan(mkv_ctx* c, int plan, int units, const int32_t* unit_lens, cudaStream_t st) {
    // Launches of one layer leave part of the SMs' CTA slots to the launch that runs alongside
    // (the next layer's, see Params::defer); a launch over several layers is never followed by
    // one that could, and takes them all.
    const int n_max = plan < c->layers ? std::max(1, (int)((long long)c->n_ctas_max * c->grid_share / 100)) : c->n_ctas_max;
    const StartTable T = build_start_table(units, c->budget_max, unit_lens, n_max, c->head_tiles,
                                           (c->flags & MKV_FLAG_REPRODUCIBLE) != 0);
    c->n_ctas[plan] = T.n_ctas;
    uint8_t* pb = plan_base(c, plan);
    const PlanOff& po = plan_off(c, plan);
    const size_t U = (size_t)units, N = (size_t)T.n_ctas;
    bool ok = true;
    auto up = [&](size_t off, const std::vector<int32_t>& v, size_t n) {
        ok &= cudaMemcpyAsync(pb + off, v.data(), n * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    };
    up(po.cta_unit0, T.cta_unit0, N);
    up(po.cta_head0, T.cta_head0, N);
    up(po.cta_headn, T.cta_headn, N);
    up(po.cta_t0, T.cta_t0, N + 1);
    up(po.unit_next0, T.next0, U);
    up(po.unit_chunk, T.chunk, U);
    up(po.tile_begin, T.tile_begin, U + 1);
    up(po.unit_cta0, T.unit_cta0, U);
    up(po.next, T.next0, U);
    up(po.next + U * 4, T.next0, U);
    ok &= cudaMemsetAsync(pb + po.cnt, 0, 2 * U * 8, st) == cudaSuccess;
    ok &= cudaMemsetAsync(pb + po.launch_no, 0, (size_t)kMaxCtas * 4, st) == cudaSuccess;
    // (the host vectors are pageable: the runtime has staged them before each call returns)
    c->stepped[plan] = 0;
    return ok ? MKV_OK : MKV_ERR_CUDA;
}

// The plan for launches over layers [layer0, layer0 + n), (re)built when the range changed or
// one of its layers was prefilled since.
mkv_status ensure_stack_plan(mkv_ctx* c, int layer0, int n, cudaStream_t st) {
    if (c->stack_n == n && c->stack_layer0 == layer0) return MKV_OK;
    std::vector<int32_t> lens;
    lens.reserve((size_t)n * c->lay.units);
    for (int l = layer0; l < layer0 + n; ++l) lens.insert(lens.end(), c->lens[l].begin(), c->lens[l].end());
    c->stack_n = 0;
    const mkv_status s = upload_plan(c, c->layers, n * c->lay.units, lens.data(), st);
    if (s != MKV_OK) return s;
    c->stack_layer0 = layer0;
    c->stack_n = n;
    return MKV_OK;
}

mkv_status layers_args(const mkv_ctx* c, int layer0, int n) {
    if (!c || n < 1 || layer0 < 0 || layer0 > c->layers - n) return MKV_ERR_INVALID_ARG;
    for (int l = layer0; l < layer0 + n; ++l)
        if (!c->prefilled[l]) return MKV_ERR_BAD_STATE;
    return MKV_OK;
}

}  // namespace

extern "C" {

size_t mkv_workspace_bytes(int layers, int batch, int q_heads, int kv_heads, int head_dim, int budget,
                           int max_prefill, int kv_dtype, int score_mode) {
    (void)score_mode;
    Layout L;
    if (!make_layout(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill, kv_dtype, &L)) return 0;
    return L.total;
}

int mkv_grid_limit(int sm_count, int resident_per_sm, int wanted_per_sm) {
    if (sm_count < 1 || resident_per_sm < 1 || wanted_per_sm < 1) return 0;
    return (int)std::min<long long>(kMaxCtas, (long long)sm_count * std::min(resident_per_sm, wanted_per_sm));
}

mkv_status mkv_plan_starts(int batch, int kv_heads, int budget, const int32_t* prefill_lens, int n_ctas_max,
                           int head_tiles, int32_t* n_ctas, int32_t* cta_unit0, int32_t* cta_head0,
                           int32_t* cta_headn, int32_t* unit_next0, int32_t* unit_chunk) {
    if (batch < 1 || kv_heads < 1 || budget < 1 || !prefill_lens || n_ctas_max < 1 || n_ctas_max > kMaxCtas)
        return MKV_ERR_INVALID_ARG;
    if (head_tiles < 0 || head_tiles > kMaxHeadTiles) return MKV_ERR_INVALID_ARG;
    if (!n_ctas || !cta_unit0 || !cta_head0 || !cta_headn || !unit_next0 || !unit_chunk) return MKV_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (prefill_lens[b] < 0) return MKV_ERR_INVALID_ARG;
    std::vector<int32_t> ul((size_t)batch * kv_heads);
    for (size_t u = 0; u < ul.size(); ++u) ul[u] = prefill_lens[u / kv_heads];
    const StartTable T = build_start_table(batch * kv_heads, budget, ul.data(), n_ctas_max, head_tiles, false);
    const size_t n = (size_t)T.n_ctas;
    *n_ctas = T.n_ctas;
    std::memcpy(cta_unit0, T.cta_unit0.data(), sizeof(int32_t) * n);
    std::memcpy(cta_head0, T.cta_head0.data(), sizeof(int32_t) * n);
    std::memcpy(cta_headn, T.cta_headn.data(), sizeof(int32_t) * n);
    std::memcpy(unit_next0, T.next0.data(), sizeof(int32_t) * T.next0.size());
    std::memcpy(unit_chunk, T.chunk.data(), sizeof(int32_t) * T.chunk.size());
    return MKV_OK;
}

mkv_status mkv_plan_ranges(int batch, int kv_heads, int budget, const int32_t* prefill_lens, int n_ctas_max,
                           int32_t* n_ctas, int32_t* cta_t0, int32_t* tile_begin, int32_t* unit_cta0) {
    if (batch < 1 || kv_heads < 1 || budget < 1 || !prefill_lens || n_ctas_max < 1 || n_ctas_max > kMaxCtas)
        return MKV_ERR_INVALID_ARG;
    if (!n_ctas || !cta_t0 || !tile_begin || !unit_cta0) return MKV_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (prefill_lens[b] < 0) return MKV_ERR_INVALID_ARG;
    std::vector<int32_t> ul((size_t)batch * kv_heads);
    for (size_t u = 0; u < ul.size(); ++u) ul[u] = prefill_lens[u / kv_heads];
    const StartTable T = build_start_table(batch * kv_heads, budget, ul.data(), n_ctas_max, 0, true);
    *n_ctas = T.n_ctas;
    std::memcpy(cta_t0, T.cta_t0.data(), sizeof(int32_t) * T.cta_t0.size());
    std::memcpy(tile_begin, T.tile_begin.data(), sizeof(int32_t) * T.tile_begin.size());
    std::memcpy(unit_cta0, T.unit_cta0.data(), sizeof(int32_t) * T.unit_cta0.size());
    return MKV_OK;
}

size_t mkv_kv_bytes_per_token(int layers, int kv_heads, int head_dim, int kv_dtype) {
    if (layers < 1 || kv_heads < 1 || head_dim < 1 || (kv_dtype != MKV_BF16 && kv_dtype != MKV_F32)) return 0;
    return (size_t)layers * kv_heads * 2 * head_dim * elem_size(kv_dtype);
}

mkv_status mkv_create(int layers, int q_heads, int kv_heads, int head_dim, int budget, float beta, int batch,
                      int max_prefill, int kv_dtype, int out_dtype, int score_mode, int kernel, unsigned flags,
                      void* workspace, size_t workspace_bytes, int device, mkv_ctx** out_ctx) {
    if (!out_ctx) return MKV_ERR_INVALID_ARG;
    *out_ctx = nullptr;
    Layout L;
    if (!make_layout(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill, kv_dtype, &L))
        return MKV_ERR_INVALID_ARG;
    if (!(beta >= 0.0f && beta <= 1.0f)) return MKV_ERR_INVALID_ARG;
    if (out_dtype != MKV_BF16 && out_dtype != MKV_F32) return MKV_ERR_INVALID_ARG;
    if (kv_dtype == MKV_F32 && out_dtype != MKV_F32) return MKV_ERR_INVALID_ARG;
    if (score_mode != MKV_SCORE_GROUP_MEAN && score_mode != MKV_SCORE_LAYER_MEAN) return MKV_ERR_INVALID_ARG;
    if (kernel < MKV_KERNEL_AUTO || kernel > MKV_KERNEL_MMA) return MKV_ERR_INVALID_ARG;
    if (flags & ~(MKV_FLAG_RECORD_PROBS | MKV_FLAG_INPUTS_READY | MKV_FLAG_REPRODUCIBLE)) return MKV_ERR_INVALID_ARG;
    if (!workspace || device < 0) return MKV_ERR_INVALID_ARG;
    const int G = q_heads / kv_heads;
    const bool mma_ok = mma_supported(kv_dtype, head_dim, G);
    const bool simt_ok = simt_supported(kv_dtype, head_dim, G);
    bool use_mma;
    if (kernel == MKV_KERNEL_MMA) { if (!mma_ok) return MKV_ERR_UNSUPPORTED; use_mma = true; }
    else if (kernel == MKV_KERNEL_SIMT) { if (!simt_ok) return MKV_ERR_UNSUPPORTED; use_mma = false; }
    else { if (!mma_ok && !simt_ok) return MKV_ERR_UNSUPPORTED; use_mma = mma_ok; }
    if (((uintptr_t)workspace % kAlign) != 0 || workspace_bytes < L.total) return MKV_ERR_WORKSPACE;

    DeviceGuard guard(device);
    if (!guard.ok) return MKV_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MKV_ERR_CUDA;

    mkv_ctx* c = new (std::nothrow) mkv_ctx();
    if (!c) return MKV_ERR_INVALID_ARG;
    c->layers = layers; c->batch = batch; c->q_heads = q_heads; c->kv_heads = kv_heads;
    c->head_dim = head_dim; c->group = G;
    c->budget = budget; c->budget_max = budget; c->max_prefill = max_prefill; c->beta = beta;
    c->kv_dtype = kv_dtype; c->out_dtype = out_dtype; c->score_mode = score_mode; c->kernel = kernel;
    c->flags = flags; c->device = device; c->sm_count = prop.multiProcessorCount;
    c->ws = (uint8_t*)workspace; c->lay = L;
    c->use_mma = use_mma;
    c->stages = 3;
    c->head_tiles = kHeadTiles;
    c->grid_share = (flags & MKV_FLAG_INPUTS_READY) ? 75 : 100;
    c->pdl = true;
    c->wait_ns = 2000000000ull;   // 2 s
    const mkv_status gs = size_grid(c);
    if (gs != MKV_OK) { delete c; return gs; }
    // Zero everything once: counters, tickets, status, and the pools (rows that are never
    // written must still hold finite numbers because masked rows enter 0 * v products).
    if (cudaMemset(workspace, 0, L.total) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        delete c;
        return MKV_ERR_CUDA;
    }
    c->prefilled.assign(layers, 0);
    c->stepped.assign(layers + 1, 0);
    c->n_ctas.assign(layers + 1, 0);
    c->stack_layer0 = 0; c->stack_n = 0;
    c->last_layer0 = 0; c->last_n = 0; c->scratch_set = 0; c->last_stream = nullptr;
    c->lens.assign(layers, std::vector<int32_t>((size_t)batch * kv_heads, 0));
    c->launches = 0;
    *out_ctx = c;
    return MKV_OK;
}

void mkv_destroy(mkv_ctx* ctx) { delete ctx; }

mkv_status mkv_set_option(mkv_ctx* c, int option, long long value) {
    if (!c) return MKV_ERR_INVALID_ARG;
    switch (option) {
        case MKV_OPT_RING_STAGES: {
            if (!c->use_mma) return MKV_ERR_UNSUPPORTED;
            if (value < 2 || value > mma_max_stages()) return MKV_ERR_INVALID_ARG;
            DeviceGuard guard(c->device);
            if (!guard.ok) return MKV_ERR_CUDA;
            const int old = c->stages;
            c->stages = (int)value;
            const mkv_status s = size_grid(c);
            if (s != MKV_OK) { c->stages = old; size_grid(c); return s; }
            break;
        }
        case MKV_OPT_HEAD_TILES:
            if (value < 0 || value > kMaxHeadTiles) return MKV_ERR_INVALID_ARG;
            c->head_tiles = (int)value;
            break;
        case MKV_OPT_GRID_SHARE:
            if (value < 10 || value > 100) return MKV_ERR_INVALID_ARG;
            c->grid_share = (int)value;
            break;
        case MKV_OPT_WAIT_LIMIT_US:
            if (value < 1 || value > 60000000ll) return MKV_ERR_INVALID_ARG;
            c->wait_ns = (unsigned long long)value * 1000ull;
            return MKV_OK;           // no plan depends on it
        case MKV_OPT_OVERLAP:
            if (value != 0 && value != 1) return MKV_ERR_INVALID_ARG;
            c->pdl = value != 0;
            return MKV_OK;
        default:
            return MKV_ERR_INVALID_ARG;
    }
    // the start tables depend on it: every layer has to be prefilled again
    std::fill(c->prefilled.begin(), c->prefilled.end(), 0);
    c->stack_n = 0;
    return MKV_OK;
}

mkv_status mkv_prefill(mkv_ctx* c, int layer, const void* K, const void* V, const int32_t* prefill_lens,
                       int src_rows, void* stream) {
    if (!layer_ok(c, layer) || !prefill_lens) return MKV_ERR_INVALID_ARG;
    std::vector<int32_t> ul((size_t)c->batch * c->kv_heads);
    for (size_t u = 0; u < ul.size(); ++u) ul[u] = prefill_lens[u / c->kv_heads];
    return mkv_prefill_units(c, layer, K, V, ul.data(), src_rows, stream);
}

mkv_status mkv_prefill_units(mkv_ctx* c, int layer, const void* K, const void* V, const int32_t* unit_lens,
                             int src_rows, void* stream) {
    if (!layer_ok(c, layer) || !unit_lens || src_rows < 0) return MKV_ERR_INVALID_ARG;
    if (c->score_mode == MKV_SCORE_LAYER_MEAN && c->kv_heads > 1) {
        // one importance vector per sequence only makes sense over equal prompts per KV head
        for (int u = 0; u < c->lay.units; ++u)
            if (unit_lens[u] != unit_lens[u - u % c->kv_heads]) return MKV_ERR_UNSUPPORTED;
    }
    int maxlen = 0;
    for (int u = 0; u < c->lay.units; ++u) {
        if (unit_lens[u] < 0 || unit_lens[u] > src_rows) return MKV_ERR_INVALID_ARG;
        if (unit_lens[u] > c->max_prefill) return MKV_ERR_CAPACITY;
        maxlen = std::max(maxlen, unit_lens[u]);
    }
    if (maxlen > 0 && (!K || !V)) return MKV_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const Layout& L = c->lay;
    const size_t U = (size_t)L.units;

    for (size_t u = 0; u < U; ++u) c->lens[layer][u] = unit_lens[u];
    if (c->stack_n > 0 && layer >= c->stack_layer0 && layer < c->stack_layer0 + c->stack_n) c->stack_n = 0;
    const mkv_status ps = upload_plan(c, layer, L.units, unit_lens, st);
    if (ps != MKV_OK) return ps;

    const LayerDev d = layer_dev(c, layer);
    bool ok = true;
    ok &= cudaMemcpyAsync((void*)d.unit_lp, c->lens[layer].data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    // empty decode pool, rewind counters
    ok &= cudaMemsetAsync(d.n_dec, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(d.n_prev, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(d.ev_k, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(d.unit_step, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(d.seq_ticket, 0, (size_t)c->batch * 4, st) == cudaSuccess;
    // the rows of head sums are zero between steps; a step that was cut short may have left some
    for (int set = 0; set < 2; ++set)
        ok &= cudaMemsetAsync(c->ws + L.scratch0 + L.scratch_bytes * set + L.so.head_sum, 0,
                              (size_t)L.layers * c->batch * L.lstride * 4, st) == cudaSuccess;
    if (!ok) return MKV_ERR_CUDA;
    if (maxlen > 0) {
        const long long total = (long long)U * src_rows * (L.rowb / 16);
        const int threads = 256;
        const int blocks = (int)std::min<long long>((total + threads - 1) / threads, 148 * 16);
        prefill_copy_kernel<<<blocks, threads, 0, st>>>((const uint8_t*)K, (const uint8_t*)V, d.Kp, d.Vp, d.unit_lp,
                                                        (int)U, src_rows, c->max_prefill, L.rowb);
        if (cudaGetLastError() != cudaSuccess) return MKV_ERR_CUDA;
        c->launches += 1;
    }
    c->prefilled[layer] = 1;
    return MKV_OK;
}

mkv_status mkv_decode_step(mkv_ctx* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                           void* stream) {
    if (!layer_ok(c, layer) || !q || !k_new || !v_new || !out) return MKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    const Params p = make_params(c, layer, 1, layer, q, k_new, v_new, out, kModeDecode);
    return launch_step(c, layer, layer, 1, p, (cudaStream_t)stream);
}

mkv_status mkv_decode_step_layers(mkv_ctx* c, int layer0, int n_layers, const void* q, const void* k_new,
                                  const void* v_new, void* out, void* stream) {
    if (!c || !q || !k_new || !v_new || !out) return MKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return MKV_ERR_INVALID_ARG;
    mkv_status s = layers_args(c, layer0, n_layers);
    if (s != MKV_OK) return s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    if ((s = ensure_stack_plan(c, layer0, n_layers, (cudaStream_t)stream)) != MKV_OK) return s;
    const Params p = make_params(c, layer0, n_layers, c->layers, q, k_new, v_new, out, kModeDecode);
    return launch_step(c, c->layers, layer0, n_layers, p, (cudaStream_t)stream);
}

mkv_status mkv_attend_only_layers(mkv_ctx* c, int layer0, int n_layers, const void* q, void* out, void* stream) {
    if (!c || !q || !out) return MKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out)) return MKV_ERR_INVALID_ARG;
    mkv_status s = layers_args(c, layer0, n_layers);
    if (s != MKV_OK) return s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    if ((s = ensure_stack_plan(c, layer0, n_layers, (cudaStream_t)stream)) != MKV_OK) return s;
    const Params p = make_params(c, layer0, n_layers, c->layers, q, nullptr, nullptr, out, kModeAttendOnly);
    return launch_step(c, c->layers, layer0, n_layers, p, (cudaStream_t)stream);
}

mkv_status mkv_decode_step_host(mkv_ctx* c, int layer, const void* qh, const void* kh, const void* vh, void* outh,
                                void* stream) {
    if (!layer_ok(c, layer) || !qh || !kh || !vh || !outh) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = elem_size(c->kv_dtype), os = elem_size(c->out_dtype);
    const size_t nq = (size_t)c->batch * c->q_heads * c->head_dim, nk = (size_t)c->batch * c->kv_heads * c->head_dim;
    uint8_t *dq = c->ws + c->lay.stage_q, *dk = c->ws + c->lay.stage_k, *dv = c->ws + c->lay.stage_v,
            *dout = c->ws + c->lay.stage_out;
    const uint8_t* q8 = (const uint8_t*)qh;
    const bool packed = (const uint8_t*)kh == q8 + nq * es && (const uint8_t*)vh == q8 + (nq + nk) * es;
    // Whether the GPU can reach a host buffer in place is asked once per (address, size) and
    // remembered for the life of the context.
    auto view = [&](const void* h, size_t bytes) -> void* {
        for (const PinEntry& e : c->pins)
            if (e.host == h && e.bytes == bytes) return e.dev;
        void* d = pinned_view(h, bytes);
        if (c->pins.size() >= 64) c->pins.erase(c->pins.begin());
        c->pins.push_back(PinEntry{h, bytes, d});
        return d;
    };
    bool gathered = false;
    if (((nq * es) | (nk * es)) % 16 == 0) {
        // pinned inputs: the GPU fetches them itself (see host_gather_kernel)
        HostPiece pq{nullptr, (uint4*)dq, (int)(nq * es / 16)}, pk{nullptr, (uint4*)dk, (int)(nk * es / 16)},
            pv{nullptr, (uint4*)dv, (int)(nk * es / 16)};
        if (packed) {
            pq.src = (const uint4*)view(qh, (nq + 2 * nk) * es);
            if (pq.src) { pk.src = pq.src + pq.n16; pv.src = pk.src + pk.n16; }
        } else {
            pq.src = (const uint4*)view(qh, nq * es);
            pk.src = (const uint4*)view(kh, nk * es);
            pv.src = (const uint4*)view(vh, nk * es);
        }
        if (pq.src && pk.src && pv.src) {
            const int total = pq.n16 + pk.n16 + pv.n16, threads = 256;
            host_gather_kernel<<<(total + threads - 1) / threads, threads, 0, st>>>(pq, pk, pv);
            if (cudaGetLastError() != cudaSuccess) return MKV_ERR_CUDA;
            c->launches += 1;
            gathered = true;
        }
    }
    if (gathered) {
        // nothing left to copy
    } else if (packed) {
        // q, k_new and v_new lie back to back on the host: one copy instead of three (the three
        // staging regions are adjacent and at least as large)
        dk = dq + nq * es;
        dv = dk + nk * es;
        if (cudaMemcpyAsync(dq, qh, (nq + 2 * nk) * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return MKV_ERR_CUDA;
    } else {
        if (cudaMemcpyAsync(dq, qh, nq * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return MKV_ERR_CUDA;
        if (cudaMemcpyAsync(dk, kh, nk * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return MKV_ERR_CUDA;
        if (cudaMemcpyAsync(dv, vh, nk * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return MKV_ERR_CUDA;
    }
    // Pinned host memory is visible to the GPU through the unified address space: the kernel
    // then writes `out` there itself (posted writes over the bus, complete when the kernel is)
    // and the step needs one copy operation fewer.  Pageable memory takes the staged copy.
    void* const direct = view(outh, nq * os);
    void* const kernel_out = direct ? direct : (void*)dout;
    Params p = make_params(c, layer, 1, layer, dq, dk, dv, kernel_out, kModeDecode);
    p.early_inputs = 0;   // the inputs arrive through the staging area, written by the kernel or copy just ahead
    const mkv_status s = launch_step(c, layer, layer, 1, p, st, true);
    if (s != MKV_OK) return s;
    if (!direct && cudaMemcpyAsync(outh, dout, nq * os, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MKV_ERR_CUDA;
    return MKV_OK;
}

mkv_status mkv_attend_only(mkv_ctx* c, int layer, const void* q, void* out, void* stream) {
    if (!layer_ok(c, layer) || !q || !out) return MKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out)) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    const Params p = make_params(c, layer, 1, layer, q, nullptr, nullptr, out, kModeAttendOnly);
    return launch_step(c, layer, layer, 1, p, (cudaStream_t)stream);
}

mkv_status mkv_set_budget(mkv_ctx* c, int budget) {
    if (!c || budget < 1) return MKV_ERR_INVALID_ARG;
    if (budget > c->budget_max) return MKV_ERR_CAPACITY;
    c->budget = budget;
    return MKV_OK;
}

mkv_status mkv_reset(mkv_ctx* c) {
    if (!c) return MKV_ERR_INVALID_ARG;
    std::fill(c->prefilled.begin(), c->prefilled.end(), 0);
    c->stack_n = 0;
    c->budget = c->budget_max;
    c->pins.clear();
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    if (cudaMemset(c->ws + c->lay.status, 0, 4) != cudaSuccess) return MKV_ERR_CUDA;
    return MKV_OK;
}

mkv_status mkv_status_sync(mkv_ctx* c, void* stream) {
    if (!c) return MKV_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MKV_ERR_CUDA;
    int32_t s = 0;
    if (cudaMemcpy(&s, c->ws + c->lay.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return MKV_ERR_CUDA;
    return (mkv_status)s;
}

int64_t mkv_launch_count(const mkv_ctx* c) { return c ? c->launches : 0; }

mkv_status mkv_get_grid(const mkv_ctx* c, int layer, int32_t* n_ctas, int32_t* n_ctas_max) {
    if (!c || layer < 0 || layer > c->layers || !n_ctas || !n_ctas_max) return MKV_ERR_INVALID_ARG;
    if (layer == c->layers) *n_ctas = c->stack_n > 0 ? c->n_ctas[layer] : 0;
    else *n_ctas = c->prefilled[layer] ? c->n_ctas[layer] : 0;
    *n_ctas_max = c->n_ctas_max;
    return MKV_OK;
}

mkv_status mkv_debug_inject(mkv_ctx* c, int layer, int what, int b, int g) {
    if (!layer_ok(c, layer) || b < 0 || b >= c->batch || g < 0 || g >= c->kv_heads) return MKV_ERR_INVALID_ARG;
    if (what != MKV_INJECT_LOST_TILE) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    if (!c->use_mma) return MKV_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    const LayerDev d = layer_dev(c, layer);
    debug_kernel<<<1, 1>>>(d, b * c->kv_heads + g);
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    return MKV_OK;
}

static mkv_status unit_args(mkv_ctx* c, int layer, int b, int g) {
    if (!layer_ok(c, layer) || b < 0 || b >= c->batch || g < 0 || g >= c->kv_heads) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    return MKV_OK;
}
#define MKV_D2H(dst, src, bytes) \
    do { if ((bytes) > 0 && cudaMemcpy((dst), (src), (bytes), cudaMemcpyDeviceToHost) != cudaSuccess) return MKV_ERR_CUDA; } while (0)

mkv_status mkv_get_decode_state(mkv_ctx* c, int layer, int b, int g, int32_t* n, int32_t* pos, float* score,
                                int cap) {
    mkv_status s = unit_args(c, layer, b, g);
    if (s != MKV_OK) return s;
    if (!n) return MKV_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    const LayerDev d = layer_dev(c, layer);
    const int u = b * c->kv_heads + g;
    MKV_D2H(n, d.n_dec + u, 4);
    if ((pos || score) && *n > cap) return MKV_ERR_CAPACITY;
    if (pos) MKV_D2H(pos, d.pos + (size_t)u * c->lay.lstride, (size_t)*n * 4);
    if (score) MKV_D2H(score, d.score + (size_t)u * c->lay.lstride, (size_t)*n * 4);
    return MKV_OK;
}

mkv_status mkv_get_last_evicted(mkv_ctx* c, int layer, int b, int g, int32_t* k, int32_t* pos, float* score,
                                int cap) {
    mkv_status s = unit_args(c, layer, b, g);
    if (s != MKV_OK) return s;
    if (!k) return MKV_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    const LayerDev d = layer_dev(c, layer);
    const int u = b * c->kv_heads + g;
    MKV_D2H(k, d.ev_k + u, 4);
    if ((pos || score) && *k > cap) return MKV_ERR_CAPACITY;
    if (pos) MKV_D2H(pos, d.ev_pos + (size_t)u * c->lay.cap, (size_t)*k * 4);
    if (score) MKV_D2H(score, d.ev_score + (size_t)u * c->lay.cap, (size_t)*k * 4);
    return MKV_OK;
}

mkv_status mkv_get_last_probs(mkv_ctx* c, int layer, int b, int g, int32_t* n, float* abar, int32_t* pos, int cap) {
    mkv_status s = unit_args(c, layer, b, g);
    if (s != MKV_OK) return s;
    if (!n) return MKV_ERR_INVALID_ARG;
    if (!(c->flags & MKV_FLAG_RECORD_PROBS)) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    const LayerDev d = layer_dev(c, layer);
    const int u = b * c->kv_heads + g;
    MKV_D2H(n, d.n_prev + u, 4);
    if ((abar || pos) && *n > cap) return MKV_ERR_CAPACITY;
    if (abar) MKV_D2H(abar, d.abar + (size_t)u * c->lay.cap, (size_t)*n * 4);
    if (pos) MKV_D2H(pos, d.abar_pos + (size_t)u * c->lay.cap, (size_t)*n * 4);
    return MKV_OK;
}

mkv_status mkv_recency_diagnostics(mkv_ctx* c, int layer, int window, float* mass, int32_t* count, float* curve,
                                   void* stream) {
    if (!layer_ok(c, layer) || window < 1 || !mass || !count || !curve) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer] || !(c->flags & MKV_FLAG_RECORD_PROBS)) return MKV_ERR_BAD_STATE;
    if (std::min(window, c->lay.cap) > diag_max_tokens()) return MKV_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    if (launch_diag(layer_dev(c, layer), c->lay.cap, window, mass, count, curve, (cudaStream_t)stream) != cudaSuccess)
        return MKV_ERR_CUDA;
    c->launches += 1;
    return MKV_OK;
}

mkv_status mkv_read_kv(mkv_ctx* c, int layer, int b, int g, int pool, int32_t* n, void* Kh, void* Vh,
                       int cap_tokens) {
    mkv_status s = unit_args(c, layer, b, g);
    if (s != MKV_OK) return s;
    if (!n || (pool != 0 && pool != 1) || cap_tokens < 0) return MKV_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    const LayerDev d = layer_dev(c, layer);
    const int u = b * c->kv_heads + g;
    const int rowb = c->lay.rowb;
    int count;
    size_t base;
    if (pool == 0) { count = c->lens[layer][u]; base = (size_t)u * c->max_prefill * rowb; }
    else { MKV_D2H(&count, d.n_dec + u, 4); base = (size_t)u * c->lay.cap * rowb; }
    *n = count;
    const int rows = std::min(count, cap_tokens);
    if (rows == 0 || (!Kh && !Vh)) return MKV_OK;
    std::vector<uint8_t> raw((size_t)rows * rowb);
    for (int which = 0; which < 2; ++which) {
        uint8_t* dst = (uint8_t*)(which == 0 ? Kh : Vh);
        if (!dst) continue;
        const uint8_t* src = (pool == 0 ? (which == 0 ? d.Kp : d.Vp) : (which == 0 ? d.Kd : d.Vd)) + base;
        MKV_D2H(raw.data(), src, raw.size());
        for (int r = 0; r < rows; ++r)
            for (int ch = 0; ch < rowb / 16; ++ch)
                std::memcpy(dst + (size_t)r * rowb + ch * 16, raw.data() + (size_t)r * rowb + ((ch ^ (r & 7)) * 16), 16);
    }
    return MKV_OK;
}

mkv_status mkv_get_step(mkv_ctx* c, int layer, int64_t* step) {
    if (!layer_ok(c, layer) || !step) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;
    int32_t s = 0;
    MKV_D2H(&s, layer_dev(c, layer).unit_step, 4);
    *step = s;
    return MKV_OK;
}

const char* mkv_status_string(mkv_status s) {
    switch (s) {
        case MKV_OK: return "ok";
        case MKV_ERR_INVALID_ARG: return "invalid argument";
        case MKV_ERR_BAD_STATE: return "bad state";
        case MKV_ERR_CAPACITY: return "capacity exceeded";
        case MKV_ERR_WORKSPACE: return "workspace too small or misaligned";
        case MKV_ERR_UNSUPPORTED: return "unsupported configuration";
        case MKV_ERR_CUDA: return "CUDA runtime error";
        case MKV_ERR_TIMEOUT: return "device wait timed out";
        case MKV_ERR_DEVICE_CHECK: return "device consistency check failed";
    }
    return "unknown status";
}

}  // extern "C"
