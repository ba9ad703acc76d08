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

struct LayerOff {
    size_t Kp, Vp, Kd, Vd, score, pos, n_dec, abar, abar_pos, n_prev, ev_k, ev_pos, ev_score, cta_unit0, cta_head0,
        cta_headn, unit_lp, unit_next0, unit_chunk, next, cnt, launch_no, unit_step, seq_ticket, end;
};
// Scratch that lives for one step only, shared by all layers of the context (calls on a
// context are ordered on one stream, and a step touches it only after every earlier kernel
// of the stream has completed).
struct ScratchOff { size_t logit, head_sum, part_o, part_ml, keys, list_a, list_b, end; };
struct Layout {
    int units, cap, rowb, lstride;
    size_t status, stage_q, stage_k, stage_v, stage_out, scratch0, scratch_bytes, layer0, layer_bytes, total;
    ScratchOff so;  // offsets relative to the scratch base
    LayerOff lo;    // offsets relative to the layer base
};

bool make_layout(int layers, int batch, int q_heads, int kv_heads, int head_dim, int budget, int max_prefill,
                 int kv_dtype, Layout* out) {
    if (layers < 1 || batch < 1 || q_heads < 1 || kv_heads < 1 || budget < 1 || max_prefill < 0) return false;
    if (q_heads % kv_heads) return false;
    if (head_dim != 64 && head_dim != 128) return false;
    if (kv_dtype != MKV_BF16 && kv_dtype != MKV_F32) return false;
    const int G = q_heads / kv_heads;
    if (G > 16) return false;
    if ((long long)budget + 1 > (1 << 24) || max_prefill > (1 << 24)) return false;
    Layout L;
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
    const size_t U = (size_t)L.units, C = (size_t)L.cap;
    o = 0;
    L.so.logit = take((size_t)batch * q_heads * L.lstride * 4);
    L.so.head_sum = take((size_t)batch * L.lstride * 4);   // zero from mkv_create's memset, kept zero by its users
    L.so.part_o = take(U * kMaxParts * G * head_dim * 4);
    L.so.part_ml = take(U * kMaxParts * G * 2 * 4);
    L.so.keys = take(U * C * 8);
    L.so.list_a = take(U * C * 4);
    L.so.list_b = take(U * C * 4);
    L.so.end = o;
    L.scratch_bytes = o;
    L.layer0 = L.scratch0 + L.scratch_bytes;
    o = 0;
    L.lo.Kp = take(U * max_prefill * L.rowb);
    L.lo.Vp = take(U * max_prefill * L.rowb);
    L.lo.Kd = take(U * C * L.rowb);
    L.lo.Vd = take(U * C * L.rowb);
    L.lo.score = take(U * L.lstride * 4);
    L.lo.pos = take(U * L.lstride * 4);
    L.lo.n_dec = take(U * 4);
    L.lo.abar = take(U * C * 4);
    L.lo.abar_pos = take(U * C * 4);
    L.lo.n_prev = take(U * 4);
    L.lo.ev_k = take(U * 4);
    L.lo.ev_pos = take(U * C * 4);
    L.lo.ev_score = take(U * C * 4);
    L.lo.cta_unit0 = take((size_t)kMaxCtas * 4);
    L.lo.cta_head0 = take((size_t)kMaxCtas * 4);
    L.lo.cta_headn = take((size_t)kMaxCtas * 4);
    L.lo.unit_lp = take(U * 4);
    L.lo.unit_next0 = take(U * 4);
    L.lo.unit_chunk = take(U * 4);
    L.lo.next = take(2 * U * 4);      // two copies each, alternating from launch to launch
    L.lo.cnt = take(2 * U * 8);
    L.lo.launch_no = take((size_t)kMaxCtas * 4);   // per CTA: launches since the prefill
    L.lo.unit_step = take(U * 4);
    L.lo.seq_ticket = take((size_t)batch * 4);
    L.lo.end = o;
    L.layer_bytes = o;
    L.total = L.layer0 + L.layer_bytes * (size_t)layers;
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

int g_min_chunk = 2;   // tiles per pull of a unit's counter, lower bound (MKV_MIN_CHUNK overrides, for tuning)

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

// Start table.  A unit's rows are a sequence of 64-row tiles (prefill tiles, then decode
// tiles); the CTAs are spread over the units in proportion to the units' tile counts (a
// full decode pool assumed).  Each CTA owns kHeadTiles tiles outright at its place, if the
// unit has that many prefill tiles left to give (these can be fetched before the previous
// step has finished); everything else is handed out by the unit's counter, which
// therefore starts behind the reserved tiles.  Returns the number of CTAs (the grid).
//
// Every visit of a unit by a CTA that covers at least one tile delivers one partial, and a unit
// has room for kMaxParts of them.  Visits are bounded by the CTAs that start in the unit plus
// the successful pulls of its counter, so the table keeps the first below kMaxHome (the grid
// shrinks when few, long units would draw more) and sizes the unit's chunk -- tiles per pull --
// so that the second stays below kMaxParts - 8 - (CTAs starting there).
int build_start_table(int units, int budget, const int32_t* unit_lens, int n_ctas_max,
                      std::vector<int32_t>& lp, std::vector<int32_t>& next0, std::vector<int32_t>& chunk,
                      std::vector<int32_t>& cta_unit0, std::vector<int32_t>& cta_head0,
                      std::vector<int32_t>& cta_headn) {
    const int U = units;
    const int td = ceil_div(budget, kTileRows);
    lp.assign(U, 0);
    next0.assign(U, 0);
    std::vector<long long> tile_begin(U + 1, 0);
    for (int u = 0; u < U; ++u) {
        lp[u] = unit_lens[u];
        tile_begin[u + 1] = tile_begin[u] + ceil_div(lp[u], kTileRows) + td;
    }
    const long long t_all = tile_begin[U];
    long long t_max = 1;
    for (int u = 0; u < U; ++u) t_max = std::max(t_max, tile_begin[u + 1] - tile_begin[u]);
    // a unit of t tiles draws at most ceil(n_ctas * t / t_all) CTAs: keep that within kMaxHome
    const long long home_cap = (long long)(kMaxHome - 1) * t_all / t_max;
    const int n_ctas = (int)std::max<long long>(1, std::min<long long>(std::min<long long>(n_ctas_max, t_all / 2), home_cap));
    cta_unit0.assign(n_ctas, 0);
    cta_head0.assign(n_ctas, 0);
    cta_headn.assign(n_ctas, 0);
    int u = 0;
    for (int cta = 0; cta < n_ctas; ++cta) {
        const long long t0 = t_all * cta / n_ctas;
        while (tile_begin[u + 1] <= t0) ++u;
        cta_unit0[cta] = u;
        if (next0[u] + kHeadTiles <= ceil_div(lp[u], kTileRows)) {
            cta_head0[cta] = next0[u];
            cta_headn[cta] = kHeadTiles;
            next0[u] += kHeadTiles;
        }
    }
    std::vector<int> home(U, 0);
    for (int cta = 0; cta < n_ctas; ++cta) home[cta_unit0[cta]] += 1;
    chunk.assign(U, 2);
    for (int u = 0; u < U; ++u) {
        const int pulls = kMaxParts - 8 - std::min(home[u], kMaxHome);     // >= 24
        const int t = (int)(tile_begin[u + 1] - tile_begin[u]) - next0[u]; // tiles the counter hands out
        chunk[u] = std::max(g_min_chunk, ceil_div(std::max(t, 1), pulls));
    }
    return n_ctas;
}

}  // namespace

struct mkv_ctx {
    int layers, batch, q_heads, kv_heads, head_dim, group;
    int budget, budget_max, max_prefill;
    float beta;
    int kv_dtype, out_dtype, score_mode, kernel;
    unsigned flags;
    int device;
    uint8_t* ws;
    Layout lay;
    int n_ctas_max; // persistent grid upper bound (SM count x resident CTAs per SM)
    bool use_mma;
    std::vector<char> prefilled;
    std::vector<char> stepped;   // a step has run on the layer since its prefill
    bool pdl;
    std::vector<int> n_ctas;
    std::vector<std::vector<int32_t>> lens;   // per layer, per (sequence, KV head) unit
    int64_t launches;
    bool direct_out;   // mkv_decode_step_host may let the kernel write pinned host memory (MKV_NO_DIRECT_OUT=1: never)
};

namespace {

LayerDev layer_dev(const mkv_ctx* c, int layer) {
    uint8_t* base = c->ws + c->lay.layer0 + c->lay.layer_bytes * (size_t)layer;
    uint8_t* sb = c->ws + c->lay.scratch0;
    const LayerOff& o = c->lay.lo;
    const ScratchOff& so = c->lay.so;
    const size_t U = (size_t)c->lay.units;
    LayerDev d;
    d.Kp = base + o.Kp; d.Vp = base + o.Vp; d.Kd = base + o.Kd; d.Vd = base + o.Vd;
    d.score = (float*)(base + o.score);
    d.pos = (int32_t*)(base + o.pos);
    d.n_dec = (int32_t*)(base + o.n_dec);
    d.logit = (float*)(sb + so.logit);
    d.head_sum = (float*)(sb + so.head_sum);
    d.abar = (c->flags & MKV_FLAG_RECORD_PROBS) ? (float*)(base + o.abar) : nullptr;
    d.abar_pos = (int32_t*)(base + o.abar_pos);
    d.n_prev = (int32_t*)(base + o.n_prev);
    d.ev_k = (int32_t*)(base + o.ev_k);
    d.ev_pos = (int32_t*)(base + o.ev_pos);
    d.ev_score = (float*)(base + o.ev_score);
    d.n_units = c->lay.units;
    d.n_ctas = c->n_ctas[layer];
    d.cta_unit0 = (const int32_t*)(base + o.cta_unit0);
    d.cta_head0 = (const int32_t*)(base + o.cta_head0);
    d.cta_headn = (const int32_t*)(base + o.cta_headn);
    d.unit_lp = (const int32_t*)(base + o.unit_lp);
    d.unit_next0 = (const int32_t*)(base + o.unit_next0);
    d.unit_chunk = (const int32_t*)(base + o.unit_chunk);
    d.next = (int32_t*)(base + o.next);
    d.cnt = (int2*)(base + o.cnt);
    d.launch_no = (uint32_t*)(base + o.launch_no);
    d.part_o = (float*)(sb + so.part_o);
    d.part_ml = (float*)(sb + so.part_ml);
    d.unit_step = (int32_t*)(base + o.unit_step);
    d.seq_ticket = (int32_t*)(base + o.seq_ticket);
    d.keys = (unsigned long long*)(sb + so.keys);
    d.list_a = (int32_t*)(sb + so.list_a);
    d.list_b = (int32_t*)(sb + so.list_b);
    return d;
}

Params make_params(const mkv_ctx* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                   int mode) {
    Params p;
    p.L = layer_dev(c, layer);
    p.q = q; p.k_new = k_new; p.v_new = v_new; p.out = out;
    p.status = (int32_t*)(c->ws + c->lay.status);
    p.batch = c->batch; p.q_heads = c->q_heads; p.kv_heads = c->kv_heads; p.group = c->group;
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
    return p;
}

mkv_status launch_step(mkv_ctx* c, int layer, const Params& p, cudaStream_t st) {
    // The first step after a prefill must see the prefill's copies complete before it reads
    // the pool; later steps may overlap their start with the previous kernel's end.
    const bool overlap = c->pdl && c->stepped[layer];
    cudaError_t e = c->use_mma ? launch_mma(p, st, overlap) : launch_simt(p, c->kv_dtype, st);
    if (e != cudaSuccess) return MKV_ERR_CUDA;
    c->launches += 1;
    c->stepped[layer] = 1;
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

}  // namespace

extern "C" {

size_t mkv_workspace_bytes(int layers, int batch, int q_heads, int kv_heads, int head_dim, int budget,
                           int max_prefill, int kv_dtype, int score_mode) {
    (void)score_mode;
    Layout L;
    if (!make_layout(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill, kv_dtype, &L)) return 0;
    return L.total;
}

mkv_status mkv_plan_starts(int batch, int kv_heads, int budget, const int32_t* prefill_lens, int n_ctas_max,
                           int32_t* n_ctas, int32_t* cta_unit0, int32_t* cta_head0, int32_t* cta_headn,
                           int32_t* unit_next0, int32_t* unit_chunk) {
    if (batch < 1 || kv_heads < 1 || budget < 1 || !prefill_lens || n_ctas_max < 1 || n_ctas_max > kMaxCtas)
        return MKV_ERR_INVALID_ARG;
    if (!n_ctas || !cta_unit0 || !cta_head0 || !cta_headn || !unit_next0 || !unit_chunk) return MKV_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (prefill_lens[b] < 0) return MKV_ERR_INVALID_ARG;
    std::vector<int32_t> lp, next0, ch, u0, h0, hn, ul((size_t)batch * kv_heads);
    for (size_t u = 0; u < ul.size(); ++u) ul[u] = prefill_lens[u / kv_heads];
    const int n = build_start_table(batch * kv_heads, budget, ul.data(), n_ctas_max, lp, next0, ch, u0, h0, hn);
    *n_ctas = n;
    std::memcpy(cta_unit0, u0.data(), sizeof(int32_t) * (size_t)n);
    std::memcpy(cta_head0, h0.data(), sizeof(int32_t) * (size_t)n);
    std::memcpy(cta_headn, hn.data(), sizeof(int32_t) * (size_t)n);
    std::memcpy(unit_next0, next0.data(), sizeof(int32_t) * next0.size());
    std::memcpy(unit_chunk, ch.data(), sizeof(int32_t) * ch.size());
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
    if (flags & ~MKV_FLAG_RECORD_PROBS) return MKV_ERR_INVALID_ARG;
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
    if (use_mma && mma_configure() != cudaSuccess) return MKV_ERR_CUDA;
    // Zero everything once: counters, tickets, status, and the pools (rows that are never
    // written must still hold finite numbers because masked rows enter 0 * v products).
    if (cudaMemset(workspace, 0, L.total) != cudaSuccess) return MKV_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return MKV_ERR_CUDA;

    mkv_ctx* c = new (std::nothrow) mkv_ctx();
    if (!c) return MKV_ERR_INVALID_ARG;
    c->layers = layers; c->batch = batch; c->q_heads = q_heads; c->kv_heads = kv_heads;
    c->head_dim = head_dim; c->group = G;
    c->budget = budget; c->budget_max = budget; c->max_prefill = max_prefill; c->beta = beta;
    c->kv_dtype = kv_dtype; c->out_dtype = out_dtype; c->score_mode = score_mode; c->kernel = kernel;
    c->flags = flags; c->device = device; c->ws = (uint8_t*)workspace; c->lay = L;
    c->use_mma = use_mma;
    int per_sm = use_mma ? 2 : 8;
    if (const char* e = std::getenv("MKV_CTAS_PER_SM")) per_sm = std::max(1, std::min(16, std::atoi(e)));
    c->n_ctas_max = std::min(kMaxCtas, prop.multiProcessorCount * per_sm);
    c->prefilled.assign(layers, 0);
    c->stepped.assign(layers, 0);
    c->pdl = true;
    if (const char* e = std::getenv("MKV_NO_OVERLAP")) c->pdl = std::atoi(e) == 0;
    c->direct_out = true;
    if (const char* e = std::getenv("MKV_NO_DIRECT_OUT")) c->direct_out = std::atoi(e) == 0;
    if (const char* e = std::getenv("MKV_MIN_CHUNK")) g_min_chunk = std::max(1, std::min(64, std::atoi(e)));
    c->n_ctas.assign(layers, 0);
    c->lens.assign(layers, std::vector<int32_t>((size_t)batch * kv_heads, 0));
    c->launches = 0;
    *out_ctx = c;
    return MKV_OK;
}

void mkv_destroy(mkv_ctx* ctx) { delete ctx; }

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
    const int U = L.units;

    std::vector<int32_t> lp, next0, chunk, cta_unit0, cta_head0, cta_headn;
    const int n_ctas = build_start_table(U, c->budget_max, unit_lens, c->n_ctas_max, lp, next0, chunk,
                                         cta_unit0, cta_head0, cta_headn);
    c->n_ctas[layer] = n_ctas;
    for (int u = 0; u < U; ++u) c->lens[layer][u] = unit_lens[u];

    uint8_t* base = c->ws + L.layer0 + L.layer_bytes * (size_t)layer;
    bool ok = true;
    ok &= cudaMemcpyAsync(base + L.lo.cta_unit0, cta_unit0.data(), (size_t)n_ctas * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.cta_head0, cta_head0.data(), (size_t)n_ctas * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.cta_headn, cta_headn.data(), (size_t)n_ctas * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.unit_lp, lp.data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.unit_next0, next0.data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.unit_chunk, chunk.data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.next, next0.data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + L.lo.next + (size_t)U * 4, next0.data(), U * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.cnt, 0, 2 * (size_t)U * 8, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.launch_no, 0, (size_t)kMaxCtas * 4, st) == cudaSuccess;
    // empty decode pool, rewind counters
    ok &= cudaMemsetAsync(base + L.lo.n_dec, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.n_prev, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.ev_k, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.unit_step, 0, U * 4, st) == cudaSuccess;
    ok &= cudaMemsetAsync(base + L.lo.seq_ticket, 0, (size_t)c->batch * 4, st) == cudaSuccess;
    if (!ok) return MKV_ERR_CUDA;
    // host vectors above are pageable: the runtime has staged them before returning
    if (maxlen > 0) {
        const long long total = (long long)U * src_rows * (L.rowb / 16);
        const int threads = 256;
        const int blocks = (int)std::min<long long>((total + threads - 1) / threads, 148 * 16);
        prefill_copy_kernel<<<blocks, threads, 0, st>>>((const uint8_t*)K, (const uint8_t*)V, base + L.lo.Kp,
                                                        base + L.lo.Vp, (const int32_t*)(base + L.lo.unit_lp), U,
                                                        src_rows, c->max_prefill, L.rowb);
        if (cudaGetLastError() != cudaSuccess) return MKV_ERR_CUDA;
        c->launches += 1;
    }
    c->prefilled[layer] = 1;
    c->stepped[layer] = 0;
    return MKV_OK;
}

mkv_status mkv_decode_step(mkv_ctx* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                           void* stream) {
    if (!layer_ok(c, layer) || !q || !k_new || !v_new || !out) return MKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return MKV_ERR_INVALID_ARG;
    if (!c->prefilled[layer]) return MKV_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MKV_ERR_CUDA;
    const Params p = make_params(c, layer, q, k_new, v_new, out, kModeDecode);
    return launch_step(c, layer, p, (cudaStream_t)stream);
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
    bool gathered = false;
    if (c->direct_out && ((nq * es) | (nk * es)) % 16 == 0) {
        // pinned inputs: the GPU fetches them itself (see host_gather_kernel)
        HostPiece pq{nullptr, (uint4*)dq, (int)(nq * es / 16)}, pk{nullptr, (uint4*)dk, (int)(nk * es / 16)},
            pv{nullptr, (uint4*)dv, (int)(nk * es / 16)};
        if (packed) {
            pq.src = (const uint4*)pinned_view(qh, (nq + 2 * nk) * es);
            if (pq.src) { pk.src = pq.src + pq.n16; pv.src = pk.src + pk.n16; }
        } else {
            pq.src = (const uint4*)pinned_view(qh, nq * es);
            pk.src = (const uint4*)pinned_view(kh, nk * es);
            pv.src = (const uint4*)pinned_view(vh, nk * es);
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
    // (Asked on every call: an address can change hands between calls.)
    void* const direct = c->direct_out ? pinned_view(outh, nq * os) : nullptr;
    void* const kernel_out = direct ? direct : (void*)dout;
    const Params p = make_params(c, layer, dq, dk, dv, kernel_out, kModeDecode);
    const mkv_status s = launch_step(c, layer, p, st);
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
    const Params p = make_params(c, layer, q, nullptr, nullptr, out, kModeAttendOnly);
    return launch_step(c, layer, p, (cudaStream_t)stream);
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
    c->budget = c->budget_max;
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
