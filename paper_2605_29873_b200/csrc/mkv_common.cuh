// Device-side data model shared by the kernels of the Moment-KV decode library.
//
// Memory model (everything lives in the caller's workspace, per layer):
//   unit u = b * kv_heads + g  -- one (sequence, KV head) pair.  Units are independent
//   (Algorithm 1 runs per layer; the GROUP score mode keeps one importance vector per KV
//   head), so a unit is the granule of scoring, selection and compaction.
//
//   Kp, Vp  [units][max_prefill][ROWB]   frozen prefill pool (Sec. 4.2 "Prefill pool")
//   Kd, Vd  [units][cap][ROWB]           decode pool, cap = largest budget + 1
//   score   [units][cap] f32             importance I_i (Eq. 5)
//   pos     [units][cap] i32             decode-step id at which the token was appended
//   n_dec   [units] i32                  tokens currently in the decode pool
// Every one of these arrays is stored for all layers back to back ([layers][units]...), so a
// run of consecutive layers is simply a longer list of units: one launch can step several
// layers at once (Algorithm 1 runs per layer and the layers' inputs are independent), with
// "sequence" index = layer * batch + sequence and unit index = layer * units + unit.
//
// A cache row is ROWB = head_dim * sizeof(element) bytes.  Rows are stored with their
// 16-byte chunks permuted: chunk c of the row in slot s sits at chunk position
// c ^ (s & 7).  Eight consecutive slots then put the same logical chunk into eight
// different 16-byte bank groups of shared memory after a straight bulk copy, which is
// what makes the ldmatrix reads of the tensor-core kernel conflict-free without any
// per-element shuffling on the way in.
//
// Work decomposition.  The rows of a unit form a sequence of 64-row tiles: the prefill
// tiles, then the decode tiles that hold rows.  Tiles are handed out per unit by an atomic
// counter, a few at a time.  Every CTA starts at its own place (CTAs are spread over the
// units in proportion to the units' tile counts, and each owns a few reserved tiles there,
// which it can fetch before anything else is known), then keeps pulling chunks of its unit
// and, when that unit is exhausted, moves on to the next unit that still has tiles.  Fast
// SMs therefore drift into the territory of slow ones and all CTAs finish together.  A CTA
// carries one online-softmax state per unit visit and delivers it as one partial
// (m, l, O[G][d]) together with the number of tiles it covered; the delivery that
// completes the unit's tile count (an atomic add, never a wait) runs that unit's tail:
// the fresh token, combine, normalised decode probabilities, head mean, momentum update,
// selection, append/compaction.  The counters exist twice and alternate from launch to
// launch; a unit's tail rewinds the idle copy, so no counter is ever reset while a CTA may
// still probe it.
//
// The fresh token of a step never travels through the streaming part: its logit, its
// probability, its importance and its row store all happen in the tail, which knows the
// evicted slot by then and writes the fresh row straight into the hole.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mkv {

constexpr int kTileRows = 64;       // rows of one tile of the work decomposition
constexpr int kMaxGroup = 8;        // G = q_heads / kv_heads the kernels are built for
constexpr int kMaxParts = 64;       // partials per unit (chunks grow to keep this)
constexpr int kMaxCtas = 2048;      // persistent grid upper bound
constexpr int kHeadTiles = 3;       // tiles a CTA owns outright at its starting place, by default (the ring's depth)
constexpr int kMaxHeadTiles = 16;   // ... and the most a context may ask for
constexpr int kHopWindow = 256;     // units a CTA looks at, ahead of its own, when its unit runs dry
constexpr int kMaxHome = 32;        // CTAs that start in one unit (bound kept by the start table)
constexpr float kNegBig = -1.0e30f; // finite stand-in for -inf in running maxima

enum : int { kModeDecode = 0, kModeAttendOnly = 1 };
enum : int { kStatusOk = 0, kStatusTimeout = 7, kStatusDeviceCheck = 8 };

struct LayerDev {
    uint8_t *Kp, *Vp, *Kd, *Vd;
    float* score;
    int32_t* pos;
    int32_t* n_dec;
    float* logit;      // [batch*q_heads][lstride] raw logits (log2 units) of decode-pool tokens
    float* head_sum;   // [batch][lstride] layer-wide score mode: per decode token the probabilities summed over
                       // all heads of the sequence (accumulated by its units' tails); all zero between steps
    float* abar;       // [units][cap] or nullptr: Eq. 4 values of the last step, slot order before its eviction
    int32_t* abar_pos; // [units][cap], with abar: the position ids of those slots
    int32_t* n_prev;   // [units] decode count (fresh token included) before the last eviction
    int32_t* ev_k;     // [units] tokens evicted by the last step
    int32_t* ev_pos;   // [units][cap]
    float* ev_score;   // [units][cap]
    int32_t n_units;
    int32_t n_ctas;             // the grid
    const int32_t* cta_unit0;   // [n_ctas] unit a CTA starts in
    const int32_t* cta_head0;   // [n_ctas] first of its reserved tiles there
    const int32_t* cta_headn;   // [n_ctas] number of reserved tiles (prefill tiles; may be 0)
    const int32_t* unit_lp;     // [units] prefill length
    const int32_t* unit_next0;  // [units] tiles reserved in the unit = start value of its counter
    const int32_t* unit_chunk;  // [units] tiles handed out per pull of the unit's counter
    // Work-sharing counters, two copies each (copy c at + c * n_units).  A launch uses the copy
    // of its own parity and its tails rewind the other one for the launch after it.  The parity
    // is found on the device: every CTA keeps, in a word of its own, the number of launches it
    // has taken part in since the layer's prefill (the grid does not change in between) -- so
    // a recorded sequence of launches (a CUDA graph) can be replayed any number of times.
    int32_t* next;     // [2][units] tiles handed out so far
    int2* cnt;         // [2][units] x: tiles delivered so far, y: partial slots taken so far
    uint32_t* launch_no;   // [kMaxCtas] launches CTA i has taken part in since the layer's prefill
    float* part_o;     // [units][kMaxParts][G][d]
    float* part_ml;    // [units][kMaxParts][G][2]  (running max in log2 units, running sum)
    int32_t* unit_step;// [units] decode steps completed
    int32_t* seq_ticket;  // [batch] KV heads of a sequence done (layer-wide score mode), zero between steps
    unsigned long long* keys;   // [units][cap] selection scratch
    int32_t* list_a;   // [units][cap] compaction scratch (holes)
    int32_t* list_b;   // [units][cap] compaction scratch (movers)
    // Reproducible mode (static partition instead of counters): the global tile sequence is cut
    // into one contiguous range per CTA.
    const int32_t* tile_begin;  // [units + 1] first global tile of a unit (full decode pool assumed)
    const int32_t* cta_t0;      // [n_ctas + 1] first global tile of a CTA's range
    const int32_t* unit_cta0;   // [units] first CTA whose range reaches into the unit
    float* unit_sum;            // [units][lstride] layer-wide score mode, reproducible: a unit's own head sums
};

struct Params {
    LayerDev L;
    const void* q;
    const void* k_new;
    const void* v_new;
    void* out;
    int32_t* status;
    int batch, q_heads, kv_heads, group, head_dim;
    int cap, max_prefill, budget;
    int lstride;       // floats per head row of the logit scratch (cap rounded up to 4)
    float beta;
    float scale_log2;  // log2(e) / sqrt(head_dim)
    int mode;
    int out_f32;
    int layer_mean;    // Eq. 4 over all heads of the layer: one score vector per sequence, shared eviction
    int launch_parity; // launches of the context so far, modulo 2 (diagnostic builds keep two trace sets)
    int early_inputs;  // the caller's q, k_new, v_new are final when the launch is enqueued: attention over
                       // reserved prompt tiles may run before the previous kernel of the stream has completed
    int defer;         // this launch shares nothing with the previous kernel of the stream (another layer, the
                       // other set of scratch, inputs final): it runs from the start and only orders its END
                       // behind the previous kernel -- every CTA passes the dependency wait before it lets
                       // the next launch begin, so launches still complete in stream order
    int det;           // reproducible mode: static partition, partial slots in CTA order
    unsigned long long wait_ns;   // limit of every bounded wait inside a kernel
};

// Parity of the launch this CTA is part of; counts the launch in the CTA's own word.  Call once
// per CTA, from one thread, after every earlier kernel of the stream has completed.  (The
// tensor-core kernel does the same by hand, with other work between the load and its use.)
__device__ inline int take_launch_parity(const LayerDev& L) {
    const uint32_t v = __ldcg(&L.launch_no[blockIdx.x]);
    L.launch_no[blockIdx.x] = v + 1u;
    return (int)(v & 1u);
}

// byte offset inside a stored row of logical byte `byte` for the row in slot `slot`
__host__ __device__ inline uint32_t swz(uint32_t slot, uint32_t byte) {
    return ((((byte >> 4) ^ (slot & 7u)) << 4) | (byte & 15u));
}

__device__ inline float to_f32(float x) { return x; }
__device__ inline float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

__device__ inline float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ inline void bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Tiles of a unit that hold rows (at least one, so that every unit is visited and its tail
// runs even when it has nothing cached yet) and the chunk handed out per pull.
__device__ inline int unit_tiles(int lp, int n_old) {
    return max(1, (lp + kTileRows - 1) / kTileRows + (n_old + kTileRows - 1) / kTileRows);
}

// Optional per-CTA timestamps (diagnostic builds only: compile with -DMKV_TRACE).  Slot i of
// CTA c is g_trace[(launch parity * kMaxCtas + c) * 16 + i]; mkv_debug_trace() copies the array
// to the host.
#ifdef MKV_TRACE
static __device__ unsigned long long g_trace[2 * kMaxCtas * 16];   // one copy per translation unit
__device__ inline unsigned long long trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define MKV_TR_AT(i) mkv::g_trace[(p.launch_parity * mkv::kMaxCtas + blockIdx.x) * 16 + (i)]
#define MKV_TR(i) (MKV_TR_AT(i) = mkv::trace_now())
#define MKV_TR_ADD(i, v) (MKV_TR_AT(i) += (v))
#define MKV_TR_SET(i, v) (MKV_TR_AT(i) = (v))
#else
#define MKV_TR(i) ((void)0)
#define MKV_TR_ADD(i, v) ((void)0)
#define MKV_TR_SET(i, v) ((void)0)
#endif

// Tile `t` of a unit's tile sequence -> (segment, first row, valid rows).  Prefill tiles
// come first; decode tiles cover the pool's rows [0, n_old).
struct TileRef { int seg, row, cnt; };
__device__ inline TileRef tile_ref(int t, int lp, int n_old) {
    const int tp = (lp + kTileRows - 1) / kTileRows;
    TileRef r;
    if (t < tp) { r.seg = 0; r.row = t * kTileRows; r.cnt = min(kTileRows, lp - r.row); }
    else { r.seg = 1; r.row = (t - tp) * kTileRows; r.cnt = max(0, min(kTileRows, n_old - r.row)); }
    return r;
}

}  // namespace mkv
