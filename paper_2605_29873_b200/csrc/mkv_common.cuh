// Device-side data model shared by the kernels of the Moment-KV decode library.
//
// Memory model (everything lives in the caller's workspace, per layer):
//   unit u = b * kv_heads + g  -- one (sequence, KV head) pair.  Units are independent
//   (Algorithm 1 runs per layer; the GROUP score mode keeps one importance vector per KV
//   head), so a unit is the granule of scoring, selection and compaction.
//
//   Kp, Vp  [units][max_prefill][ROWB]   frozen prefill pool (Sec. 4.2 "Prefill pool")
//   Kd, Vd  [units][cap][ROWB]           decode pool, cap = largest budget + 1 (the fresh
//                                        token sits in the pool during its own step)
//   score   [units][cap] f32             importance I_i (Eq. 5)
//   pos     [units][cap] i32             decode-step id at which the token was appended
//   n_dec   [units] i32                  tokens currently in the decode pool
//
// A cache row is ROWB = head_dim * sizeof(element) bytes.  Rows are stored with their
// 16-byte chunks permuted: chunk c of the row in slot s sits at chunk position
// c ^ (s & 7).  Eight consecutive slots then put the same logical chunk into eight
// different 16-byte bank groups of shared memory after a straight bulk copy, which is
// what makes the ldmatrix reads of the tensor-core kernel conflict-free without any
// per-element shuffling on the way in.
//
// Work decomposition: the rows of every unit (prefill segment, then decode segment up to
// cap) are cut into "items" of at most item_rows rows; an item never straddles the two
// segments.  An item yields one partial (m, l, O[G][d]) of the online softmax.  The last
// CTA to deliver a partial of a unit (an atomic ticket, never a wait) runs that unit's
// tail: combine, normalise the decode probabilities, head mean, momentum update,
// selection, compaction.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mkv {

constexpr int kMaxGroup = 16;       // G = q_heads / kv_heads
constexpr int kMaxParts = 128;      // partials per unit (item_rows grows to keep this)
constexpr float kNegBig = -1.0e30f; // finite stand-in for -inf in running maxima

enum : int { kModeDecode = 0, kModeAttendOnly = 1 };
enum : int { kStatusOk = 0, kStatusTimeout = 7, kStatusDeviceCheck = 8 };

struct Item {          // 16 bytes, read as one int4
    int32_t unit;
    int32_t row0;      // first row inside the segment
    int32_t rows;      // rows covered (decode segment: of the capacity range)
    int32_t seg;       // 0 prefill, 1 decode
};

struct LayerDev {
    uint8_t *Kp, *Vp, *Kd, *Vd;
    float* score;
    int32_t* pos;
    int32_t* n_dec;
    float* logit;      // [batch*q_heads][cap] raw logits (log2 units) of decode tokens
    float* abar;       // [units][cap] or nullptr
    int32_t* n_prev;   // [units] decode count before the last eviction
    int32_t* ev_k;     // [units] tokens evicted by the last step
    int32_t* ev_pos;   // [units][cap]
    float* ev_score;   // [units][cap]
    const Item* items;
    int32_t n_items;
    const int32_t* unit_lp;     // [units] prefill length
    const int32_t* unit_part0;  // [units] first item (= partial) index of the unit
    const int32_t* unit_nparts; // [units]
    float* part_o;     // [n_items][G][d]
    float* part_ml;    // [n_items][G][2]  (running max in log2 units, running sum)
    int32_t* ticket;   // [units]
    int32_t* sched;    // [0] work counter  [1] CTAs done
    int32_t* step;     // [1] decode steps completed
    unsigned long long* keys;   // [units][cap] selection scratch
    int32_t* list_a;   // [units][cap] compaction scratch (holes)
    int32_t* list_b;   // [units][cap] compaction scratch (movers)
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
    float beta;
    float scale_log2;  // log2(e) / sqrt(head_dim)
    int mode;
    int out_f32;
};

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

// Last CTA out of the kernel rewinds the scheduler words and advances the step counter.
__device__ inline void grid_epilogue(const Params& p, unsigned n_ctas) {
    __threadfence();
    const int prev = atomicAdd(&p.L.sched[1], 1);
    if (prev == (int)n_ctas - 1) {
        p.L.sched[0] = 0;
        p.L.sched[1] = 0;
        if (p.mode == kModeDecode) p.L.step[0] = p.L.step[0] + 1;
        __threadfence();
    }
}

}  // namespace mkv
