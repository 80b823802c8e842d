// TLI verification for sm_100a: kernels and the C ABI declared in include/tli.h.
//
// A call is two launches (four for vocabularies or batches too large for the cluster kernel).
// The passes over logits are HBM-bound; there is no dense contraction on this path, hence no
// tensor cores.
//
//   tli_stats_kernel   persistent grid, two CTAs per SM, each one producer warp and sixteen
//                      consumer warps around a 96 KB ring of shared-memory stages filled by
//                      cp.async.bulk with mbarrier completion.  Target rows: (reference, sum of
//                      2^(z*s - reference)) with s = log2(e)/tau; drafter rows: the same over ids
//                      inside the intersection only (Algorithm 4's renormalisation: the
//                      full-softmax denominator cancels in q' = q / sum_{T cap D} q);
//                      temperature-0 rows: (max, lowest index).  One pair per segment of a row
//                      goes to the workspace.
//   tli_finish_kernel  one thread-block cluster per sequence: fp64 combination of the pairs,
//                      Algorithm 5's acceptance tests and count of accepted drafts, then the extra
//                      token: the drafter row staged in shared memory, weights max(0, p - q'_T)
//                      (or p for the bonus row) over the CTAs' slices of the one target row, the
//                      CDF inverted through distributed shared memory.
//   tli_decide_kernel, tli_sample_kernel, tli_select_kernel
//                      the same in three kernels for rows that do not fit a cluster's shared
//                      memory: decision per sequence, one CTA per 16 KB tile of the target row
//                      (q'_T gathered through the inverse map), inversion tile -> vector -> element.
//
// Beside the verification call: tli_draft_kernel / tli_draft_select_kernel draw one id per row of
// logits by inverse CDF (the drafts from q' for tli_draft_sample; with no mask, the target tokens
// of Algorithm 2 for tli_slem_verify, compared by tli_slem_match_kernel), tli_rate_*_kernel form
// the paper's expected acceptance rates per draft position (tli_acceptance_rates), and
// tli_shard_*_kernel are the local steps of the verification over vocabulary shards.
//
// Softmax terms are formed as ex2(fma(z, s, -c)) with an integer-valued reference c in log2
// units: the only per-term rounding is the one in the fma, and every change or combination of
// references is an exact power of two.

#include <cuda_runtime.h>
#include <float.h>
#include <limits.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <mutex>
#include <new>
#include <vector>

#include "tli.h"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kVecPerThread = 4;
constexpr int kVecPerTile = kThreads * kVecPerThread;       // sampling pass: 1024 16-byte vectors per tile
constexpr int kTileBytes = kVecPerTile * 16;                // 16 KB
constexpr int kRingBytes = 96 * 1024;                       // shared-memory stage ring of the statistics kernel
constexpr int kMaxStages = 12;
constexpr int kCtasPerSm = 2;                               // persistent CTAs of the statistics kernel per SM
constexpr int kSWarps = 16;                                 // consumer warps of the statistics kernel
constexpr int kSThreads = kSWarps * 32;
constexpr int kMaxTiles = (TLI_MAX_V * 4 + 15) / kTileBytes + 2;
constexpr float kNegBig = -FLT_MAX;

enum : int { MODE_SKIP = 0, MODE_RESIDUAL = 1, MODE_TARGET_ONLY = 2 };

struct __align__(16) RowSel {   // what the sampling pass needs for one sequence
    int n;               // accepted drafts = row to sample from
    int mode;            // MODE_*
    float s;             // log2(e) / tau
    float c_t;           // reference of target row n (log2 units)
    float rs_t;          // 1 / sum of target row n
    float c_d;           // reference of drafter row n
    float rs_d;          // 1 / intersection sum of drafter row n (0 if empty)
    float v;             // uniforms[b, K]
};

// Division of a 32-bit number by a divisor fixed on the host: q = (mulhi(n, m) + n) >> s with
// s = ceil(log2 d) and m = floor(2^32 (2^s - d) / d) + 1, exact for every 32-bit n (the sum is
// formed in 64 bits).  The producer thread of the statistics kernel decodes every segment number
// with three of these instead of three hardware-less divisions of ~100 instructions.
struct FastDiv {
    unsigned m, s, d;
};

struct Params {
    int B, K, V_t, V_d;
    const void *zt; long long t_sb, t_sk;
    const void *zd; long long d_sb, d_sk;
    const int *map; const int *inv; const uint32_t *maskbits; int n_mapped;
    const int *draft; const float *tau; const float *u;
    const int *draft_len;    // NULL, or per sequence how many of its K drafts count (three-kernel form only)
    int *accepted; int *next_token; int *status; float *p_out; float *q_out;
    float2 *part_t; float2 *part_d; RowSel *sel; double *tilesum;
    unsigned *cnt_stats; unsigned *cnt_sample;
    unsigned *error;     // sticky: set when a bounded wait ran out
    unsigned long long *seg_counter;    // segment scheduler of the statistics kernel: segments taken from the front (low
                                        // half) and from the back (high half); zero between calls
    unsigned *cta_done;                 // ... and the CTAs that have left
    int ntile;           // 16 KB tiles per target row (sampling pass)
    int split_select;    // 1: the CDF inversions run as a kernel of their own
    int seg_vec;         // statistics kernel: 16-byte vectors per segment
    int nst, nsd;        // ... and segments per target / drafter row
    FastDiv div_per_b, div_nst, div_nsd;   // by the segments of a sequence, of a target row, of a drafter row
    // vocabulary-sharded calls (all zero otherwise): V_t / V_d above are the widths of this shard's
    // slices, which hold target ids t_begin .. and drafter ids d_begin ..; map, inv and the mask are
    // indexed by global ids
    int t_begin, d_begin;
    int sh_wd;           // drafter ids per shard (the gathered rows of shard g start at g * sh_stride elements)
    long long sh_stride;
    double *tilesum_p;   // tile sums of p beside those of the residual
    int poll_parts;      // cluster kernel: the partials lie in the context's own buffer, which holds kPartEmpty wherever no
                         // call is under way, and are waited for one by one (see tli_finish_kernel)
    int early_trigger;   // ... and the statistics grid leaves SMs free: the cluster kernel may become resident at once
    int fin_slice;       // cluster kernel: 16-byte vectors of the sampled target row per CTA
    int fin_dvec;        // cluster kernel: 16-byte vectors reserved for the staged drafter row
};

// ---------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ int float_order(float f) {       // monotone float -> int
    int i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float order_float(int i) {
    return __int_as_float(i ^ ((i >> 31) & 0x7fffffff));
}
__device__ __forceinline__ float warp_max(float m) {
    return order_float(__reduce_max_sync(0xffffffffu, float_order(m)));
}
__device__ __forceinline__ double warp_sum(double s) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

template <int DT> struct Elt;
template <> struct Elt<TLI_F32> {
    static constexpr int kBytes = 4;
    static constexpr int kPerVec = 4;
    static constexpr uint32_t kNegInfWord = 0xff800000u;
};
template <> struct Elt<TLI_BF16> {
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
    static constexpr uint32_t kNegInfWord = 0xff80ff80u;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int DT> __device__ __forceinline__ float load_elt(const void *row, long long i) {
    // (single elements are gathered: they go past L1, which the coalesced loads of the same kernels need)
    if (DT == TLI_F32) return __ldcg(reinterpret_cast<const float *>(row) + i);
    return __uint_as_float(static_cast<uint32_t>(__ldcg(reinterpret_cast<const unsigned short *>(row) + i)) << 16);
}

template <int DT> __device__ __forceinline__ void unpack(const uint4 &r, float (&z)[Elt<DT>::kPerVec]) {
    if constexpr (DT == TLI_F32) {
        z[0] = __uint_as_float(r.x); z[1] = __uint_as_float(r.y);
        z[2] = __uint_as_float(r.z); z[3] = __uint_as_float(r.w);
    } else {
        z[0] = bf16_lo(r.x); z[1] = bf16_hi(r.x); z[2] = bf16_lo(r.y); z[3] = bf16_hi(r.y);
        z[4] = bf16_lo(r.z); z[5] = bf16_hi(r.z); z[6] = bf16_lo(r.w); z[7] = bf16_hi(r.w);
    }
}

// A logit row seen as 16-byte vectors on the aligned address grid.  Vector v
// holds elements [v*EPV - head, v*EPV - head + EPV); elements outside [0, V)
// read as -inf.
template <int DT> struct RowView {
    const uint4 *vec0;   // 16-byte aligned address at or below the row start
    const void *row;     // the row itself
    int head;            // elements of vector 0 that precede the row
    int V;
    __device__ RowView(const void *base, long long elem_off, int V_) {
        const char *p = reinterpret_cast<const char *>(base) + elem_off * Elt<DT>::kBytes;
        uintptr_t a = reinterpret_cast<uintptr_t>(p);
        uintptr_t a0 = a & ~static_cast<uintptr_t>(15);
        vec0 = reinterpret_cast<const uint4 *>(a0);
        row = p;
        head = static_cast<int>(a - a0) / Elt<DT>::kBytes;
        V = V_;
    }
    __device__ __forceinline__ int first_elem(int v) const { return v * Elt<DT>::kPerVec - head; }
    __device__ __forceinline__ int nvec() const { return (V + head + Elt<DT>::kPerVec - 1) / Elt<DT>::kPerVec; }
    // Whole vectors with one 128-bit load; the two ragged ends element by element.
    __device__ __forceinline__ uint4 load(int v) const {
        const int e0 = first_elem(v);
        if (e0 >= 0 && e0 + Elt<DT>::kPerVec <= V) return __ldg(vec0 + v);
        uint32_t w[4] = {Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord};
        if constexpr (DT == TLI_F32) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int e = e0 + i;
                if (e >= 0 && e < V) w[i] = __ldg(reinterpret_cast<const uint32_t *>(row) + e);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                int e = e0 + i;
                if (e >= 0 && e < V) {
                    uint32_t h = __ldg(reinterpret_cast<const unsigned short *>(row) + e);
                    w[i >> 1] = (i & 1) ? ((w[i >> 1] & 0x0000ffffu) | (h << 16)) : ((w[i >> 1] & 0xffff0000u) | h);
                }
            }
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// bit i = 1 iff drafter id e0 + i is inside the intersection (ids outside [0, V_d) read 0;
// the bit array is zero padded by two words).
__device__ __forceinline__ uint32_t mask_bits(const uint32_t *maskbits, int e0) {
    if (e0 < 0) return __ldg(maskbits) << (-e0);
    const uint32_t lo = __ldg(maskbits + (e0 >> 5));
    const uint32_t hi = __ldg(maskbits + (e0 >> 5) + 1);
    return __funnelshift_r(lo, hi, e0 & 31);
}

// 2^d for an integer-valued d <= 0, exactly (0 below the normal range).
__device__ __forceinline__ float pow2_neg(float d) {
    return (d >= -126.f) ? __int_as_float((static_cast<int>(d) + 127) << 23) : 0.f;
}
__device__ __forceinline__ double pow2_neg_d(float d) {
    return (d >= -1022.f) ? __hiloint2double((static_cast<int>(d) + 1023) << 20, 0) : 0.0;
}
// A softmax reference for values up to m*s: the next integer above, so that every later
// change of reference is an exact power of two.  Nothing to refer to (-inf) gives kNegBig.
__device__ __forceinline__ float reference_for(float ms) { return fmaxf(ceilf(ms), kNegBig); }

// ---------------------------------------------------------------------------
// pass 1: statistics of every row, persistent and pipelined
// ---------------------------------------------------------------------------
//
// Work unit: a segment = a run of consecutive 16-byte vectors of one logit row (up to 128 KB).
// Segments are numbered sequence-major and handed out by an atomic counter to a fixed grid of CTAs.
// In each CTA one thread (the producer) streams the vectors into a ring of shared-memory stages
// with cp.async.bulk, completion counted on an mbarrier per stage; sixteen consumer warps reduce a
// stage from shared memory and hand it back through a second mbarrier as soon as its bytes are in
// registers.

// ---- mbarrier and bulk-copy primitives ----

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitLimit polls, records the fact and lets the caller go on
// (results of that call are then flagged, never trusted).  Returns false on timeout.
constexpr unsigned kWaitLimit = 1u << 22;
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, unsigned parity, int *sm_error, unsigned *g_error,
                                            unsigned limit = kWaitLimit) {
    if (*reinterpret_cast<volatile int *>(sm_error)) return false;
    for (unsigned i = 0; i < limit; ++i) {
        if (mbar_test(bar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    *reinterpret_cast<volatile int *>(sm_error) = 1;
    atomicOr(g_error, 1u);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, int *sm_error, unsigned *g_error) {
    if (mbar_test(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, sm_error, g_error);
}
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// A partial result in the context's own buffer: both words are all ones until the statistics kernel
// has stored the pair (a reference is never NaN, a sum that is NaN is the canonical positive one, an
// index is never -1).  Returns false if the pair has not arrived after kWaitLimit polls or the
// statistics kernel has given up.
constexpr uint32_t kPartEmpty = 0xffffffffu;
__device__ __forceinline__ bool load_partial_when_stored(const float2 *p, const unsigned *g_error, float2 &v) {
    for (unsigned i = 0; i < kWaitLimit; ++i) {
        asm volatile("ld.relaxed.gpu.global.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p) : "memory");
        if (__float_as_uint(v.x) != kPartEmpty && __float_as_uint(v.y) != kPartEmpty) return true;
        if ((i & 31u) == 31u && *reinterpret_cast<const volatile unsigned *>(g_error)) break;
        if (i > 4) __nanosleep(40);
    }
    return false;
}
__device__ __forceinline__ float2 ld_shared_pair(const float2 *p) {     // a pair another warp wrote: not from a register copy
    float2 v;
    asm volatile("ld.volatile.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(smem_addr(p)) : "memory");
    return v;
}

// ---- the schedule both the producer and the consumers walk ----
//
// A row is seen as 16-byte vectors on the aligned address grid (RowView).  A segment is a run of
// consecutive vectors of one row and leaves one partial result; a stage of the ring holds up to
// 512*CV vectors of it.  Segments are numbered sequence-major and handed out in that order.
// A CTA asks for its next segment only when every stage of the one before has been issued: what it
// holds when the list runs out is then its ring of stages and nothing else.  (Asking one or two
// segments ahead hides the latency of the counter and of the temperature load, but the slower CTA
// of an SM then sits on up to two more segments at the end while the others are idle: measured,
// 3 to 5 us longer on batches of a few hundred MB.)

struct Segment {
    int b;            // sequence
    int row;          // 0..K target rows, K+1..2K drafter rows
    int v0, v1;       // vectors [v0, v1) of the row's grid (clipped to the row by the producer)
    int seg;          // index of the segment within its row
    bool skip;        // nothing to read (bad temperature, or drafter row at temperature 0)
    float tau;
    int m;            // drafts of the sequence that count
};

__device__ __forceinline__ unsigned segment_count(const Params &P) {       // the host made sure it fits 32 bits
    return static_cast<unsigned>(P.B) * static_cast<unsigned>((P.K + 1) * P.nst + P.K * P.nsd);
}
__device__ __forceinline__ unsigned fast_div(unsigned n, const FastDiv &f) {
    return static_cast<unsigned>((static_cast<unsigned long long>(__umulhi(n, f.m)) + n) >> f.s);
}

// The index arithmetic of a segment, and the loads of its sequence's temperature and draft count
// (used by finish_segment()).
__device__ __forceinline__ Segment decode_segment(const Params &P, unsigned id) {
    Segment g;
    g.b = static_cast<int>(fast_div(id, P.div_per_b));
    int item = static_cast<int>(id - static_cast<unsigned>(g.b) * P.div_per_b.d);
    g.tau = __ldg(P.tau + g.b);
    g.m = P.draft_len ? __ldg(P.draft_len + g.b) : P.K;
    if (item < (P.K + 1) * P.nst) {
        g.row = static_cast<int>(fast_div(static_cast<unsigned>(item), P.div_nst)); g.seg = item - g.row * P.nst;
    } else {
        item -= (P.K + 1) * P.nst;
        const int j = static_cast<int>(fast_div(static_cast<unsigned>(item), P.div_nsd));
        g.row = P.K + 1 + j; g.seg = item - j * P.nsd;
    }
    g.v0 = g.seg * P.seg_vec;
    g.v1 = g.v0 + P.seg_vec;
    g.skip = false;
    return g;
}
__device__ __forceinline__ void finish_segment(const Params &P, Segment &g) {
    const bool bad = !(g.tau >= 0.f) || isinf(g.tau);
    const int m = min(max(g.m, 0), P.K);
    if (g.row <= P.K) g.skip = bad || g.row > m;                   // target rows 0..m: m drafts and the bonus position
    else g.skip = bad || g.tau == 0.f || g.row - P.K - 1 >= m;
}

template <int DT> __device__ __forceinline__ RowView<DT> segment_row(const Params &P, const Segment &g) {
    if (g.row <= P.K)
        return RowView<DT>(P.zt, static_cast<long long>(g.b) * P.t_sb + static_cast<long long>(g.row) * P.t_sk, P.V_t);
    return RowView<DT>(P.zd, static_cast<long long>(g.b) * P.d_sb + static_cast<long long>(g.row - P.K - 1) * P.d_sk, P.V_d);
}

// Vectors [v0, v1) of the range [a, b) that lie wholly inside the row.  Only these are bulk-copied;
// the (at most two) ragged vectors of a row are read element by element by the consumers.
template <int DT> __device__ __forceinline__ void full_vectors(const RowView<DT> &rv, int a, int b, int &v0, int &v1) {
    constexpr int EPV = Elt<DT>::kPerVec;
    const int first_full = rv.head ? 1 : 0;
    const int end_full = (rv.V + rv.head) / EPV;               // vectors [first_full, end_full) are whole
    v0 = max(a, first_full);
    v1 = min(b, end_full);
    if (v1 < v0) v1 = v0;
}

enum : int { META_FIRST = 1, META_LAST = 2, META_END = 4, META_INTERIOR = 16 };

// What the producer tells the consumers about the vectors it put into a stage: the stage holds
// vectors [v0, v0 + nv) of the row, vector v0 + i at position i.  The label also carries the
// decoded segment, so that only the producer thread divides segment numbers and reads temperatures.
struct __align__(16) StatsMeta {
    int v0, nv;
    int flags;
    int b, row;       // as in Segment
    int seg;
    float tau;
    int pad;
};

// Per-warp results of a segment wait in one of kMaxStages + 1 slots (slot = the CTA's segment
// count modulo that): a warp can be at most a ring of stages, hence at most kMaxStages segment
// ends, ahead of the warp that is still combining a slot, so no slot is rewritten while in use.
constexpr int kPairSlots = kMaxStages + 1;
struct StatsSmem {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    StatsMeta meta[kMaxStages];
    float2 pairs[kPairSlots][kSWarps];
    unsigned arrived[kPairSlots];
    int error;
};

constexpr int kStatsSmemBytes = kRingBytes + static_cast<int>(sizeof(StatsSmem));

// This thread's vectors of one stage: vector q*kSThreads + tid of the stage for q < nq.  A full
// stage that lies wholly inside the row comes straight from shared memory; a short one checks its
// length; one that touches an end of the row checks every vector.
template <int DT, int CV>
__device__ __forceinline__ void load_stage(const RowView<DT> &rv, int v0, int nv, bool interior, const uint4 *stage, int tid,
                                           uint4 (&raw)[CV]) {
    const uint4 ninf = make_uint4(Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord);
    if (interior && nv == kSThreads * CV) {
#pragma unroll
        for (int q = 0; q < CV; ++q) raw[q] = stage[q * kSThreads + tid];
    } else if (interior) {
#pragma unroll
        for (int q = 0; q < CV; ++q) {
            const int i = q * kSThreads + tid;
            raw[q] = (i < nv) ? stage[i] : ninf;
        }
    } else {
        int f0, f1;
        full_vectors<DT>(rv, v0, v0 + nv, f0, f1);
#pragma unroll
        for (int q = 0; q < CV; ++q) {
            const int i = q * kSThreads + tid;
            const int v = v0 + i;
            if (i >= nv) raw[q] = ninf;
            else if (v >= f0 && v < f1) raw[q] = stage[i];
            else raw[q] = rv.load(v);                                   // ragged end of the row
        }
    }
}

// Two fp32 lanes in one 64-bit register: the packed fma / add of sm_100, each lane rounded as the
// scalar instruction would.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_max(const uint4 &r) {
    return bf16x2_max(bf16x2_max(r.x, r.y), bf16x2_max(r.z, r.w));
}

// bf16 vectors of a drafter row: the elements whose mask bit is 0 become -inf, two at a time.
// The low eight bits of `bits` go to the top bits of eight bytes (a multiplication by four
// shifted ones, four bits per word), prmt's sign replication widens each to a 16-bit lane mask.
__device__ __forceinline__ uint32_t prmt_sign(uint32_t a, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(0u), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t keep_or_neg_inf(uint32_t w, uint32_t lanes) {
    return (w & lanes) | (~lanes & Elt<TLI_BF16>::kNegInfWord);
}
__device__ __forceinline__ void mask_bf16_vector(uint4 &r, uint32_t bits) {
    const uint32_t lo = (bits & 0xfu) * 0x10204080u;           // bit i -> top bit of byte i
    const uint32_t hi = ((bits >> 4) & 0xfu) * 0x10204080u;
    r.x = keep_or_neg_inf(r.x, prmt_sign(lo, 0x9988u));        // bytes 0,0,1,1 of lo, sign-replicated
    r.y = keep_or_neg_inf(r.y, prmt_sign(lo, 0xbbaau));        // bytes 2,2,3,3
    r.z = keep_or_neg_inf(r.z, prmt_sign(hi, 0x9988u));
    r.w = keep_or_neg_inf(r.w, prmt_sign(hi, 0xbbaau));
}

// The first nq of a thread's vectors of a stage into its running (reference, sum).  nq is the
// same for the whole CTA; FULL: the caller knows that nq == CV (no tests in the unrolled loops).
template <int DT, int CV, bool MASKED, bool FULL>
__device__ __forceinline__ void softmax_chunk(const uint4 (&raw)[CV], const uint32_t (&bits)[CV], int nq, float s,
                                              float &c_run, float &acc) {
    constexpr int EPV = Elt<DT>::kPerVec;
    // largest value of the vectors (over ids inside the intersection for a drafter row)
    float m;
    if (DT == TLI_BF16 && !MASKED) {
        uint32_t mm = bf16x2_max(raw[0]);
#pragma unroll
        for (int q = 1; q < CV; ++q)
            if (FULL || q < nq) mm = bf16x2_max(mm, bf16x2_max(raw[q]));
        m = fmaxf(bf16_lo(mm), bf16_hi(mm));
    } else {
        m = -INFINITY;
#pragma unroll
        for (int q = 0; q < CV; ++q) {
            if (!FULL && q >= nq) continue;
            float z[EPV];
            unpack<DT>(raw[q], z);
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                if (MASKED) z[i] = ((bits[q] >> i) & 1u) ? z[i] : -INFINITY;
                m = fmaxf(m, z[i]);
            }
        }
    }
    // raise the reference if these vectors top it; the sum follows by an exact power of two
    const float ms = m * s;
    if (ms > c_run) {
        const float c_new = reference_for(ms);
        acc *= pow2_neg(c_run - c_new);
        c_run = c_new;
    }
    // four running sums (elements i, i+4, i+8, ... each), two to a packed register
    const uint64_t s2 = pack2(s, s), nc2 = pack2(-c_run, -c_run);
    uint64_t a2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
    for (int q = 0; q < CV; ++q) {
        if (!FULL && q >= nq) continue;
        float z[EPV];
        unpack<DT>(raw[q], z);
#pragma unroll
        for (int i = 0; i < EPV; i += 2) {
            if (MASKED) {
                z[i] = ((bits[q] >> i) & 1u) ? z[i] : -INFINITY;
                z[i + 1] = ((bits[q] >> (i + 1)) & 1u) ? z[i + 1] : -INFINITY;
            }
            float x0, x1;
            unpack2(fma2(pack2(z[i], z[i + 1]), s2, nc2), x0, x1);
            a2[(i >> 1) & 1] = add2(a2[(i >> 1) & 1], pack2(ex2(x0), ex2(x1)));
        }
    }
    float a0, a1, a3, a4;
    unpack2(a2[0], a0, a1);
    unpack2(a2[1], a3, a4);
    acc += (a0 + a1) + (a3 + a4);
}

// Temperature-0 rows: (largest value, lowest index attaining it) over the first nq vectors.
// bf16: a running pair of packed maxima (even and odd positions) tells in five instructions
// whether a vector can raise the maximum at all; only then are its eight elements compared.  After
// every stage the pair is raised to the largest value the whole warp has seen (all of it at lower
// indices than anything the warp reads later), so that from the second stage of a segment on the
// element-wise path is rare for the warp as a whole and not just for each lane.
// In the first stage of a segment there is no such value yet: the warp first takes the largest value
// of the whole stage (packed maxima only) and lets through what reaches it -- the pair starts one
// bf16 step below it, because an equal value may be the one with the lowest index.
template <int DT, int CV, bool FULL>
__device__ __forceinline__ void argmax_chunk(const uint4 (&raw)[CV], int nq, bool first_stage, const RowView<DT> &rv,
                                             int v_first, uint32_t &mm, float &best, int &best_idx) {
    constexpr int EPV = Elt<DT>::kPerVec;
    if constexpr (DT == TLI_BF16) {
        if (first_stage) {
            uint32_t sm = bf16x2_max(raw[0]);
#pragma unroll
            for (int q = 1; q < CV; ++q)
                if (FULL || q < nq) sm = bf16x2_max(sm, bf16x2_max(raw[q]));
            const float m_w = warp_max(fmaxf(bf16_lo(sm), bf16_hi(sm)));
            const uint32_t h = __float_as_uint(order_float(float_order(m_w) - 0x10000)) >> 16;    // one step below
            mm = h | (h << 16);
        }
    }
#pragma unroll
    for (int q = 0; q < CV; ++q) {                        // increasing index order, strict > keeps the lowest
        if (!FULL && q >= nq) continue;
        if constexpr (DT == TLI_BF16) {
            const uint32_t nm = bf16x2_max(mm, bf16x2_max(raw[q]));
            if (nm == mm) continue;
            mm = nm;
        }
        float z[EPV];
        unpack<DT>(raw[q], z);
        const int e0 = rv.first_elem(v_first + q * kSThreads);
#pragma unroll
        for (int i = 0; i < EPV; ++i)
            if (z[i] > best) { best = z[i]; best_idx = e0 + i; }
    }
    if constexpr (DT == TLI_BF16) {
        const float m_w = warp_max(fmaxf(bf16_lo(mm), bf16_hi(mm)));       // a bf16 value, or -inf
        const uint32_t h = __float_as_uint(m_w) >> 16;
        mm = bf16x2_max(mm, h | (h << 16));
    }
}

// Segments are handed out by an atomic counter: a CTA that is slow simply takes fewer of them.
// The producer thread streams the vectors of its segment through the stage ring, labels every stage
// for the consumers, and then asks for the next segment (see above).
// CV = 16-byte vectors per consumer thread per stage: a stage is kSThreads*CV*16 bytes and the
// ring holds kRingBytes / that many stages.  Large batches use large stages (less bookkeeping per
// byte), small ones small stages (more parallelism across CTAs).
template <int DT, int CV>
__global__ void __launch_bounds__(kSThreads + 32, kCtasPerSm) tli_stats_kernel(const Params P) {
    constexpr int CVEC = kSThreads * CV;                       // vectors per stage
    constexpr int NST = kRingBytes / (CVEC * 16);              // stages
    static_assert(NST >= 2 && NST <= kMaxStages, "stage count");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw);
    StatsSmem &sm = *reinterpret_cast<StatsSmem *>(smem_raw + kRingBytes);
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < NST; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kSWarps); }
        for (int i = 0; i < kPairSlots; ++i) sm.arrived[i] = 0u;
        sm.error = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Launched as a programmatic dependent: when the kernel before it in the stream is the last one
    // of an earlier call (they let their dependents start at once), the CTAs of this grid are set
    // up while that call is still finishing; nothing is read or written before it has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // A small batch leaves room on the SMs: the cluster kernel, which waits for single partials and not
    // for this grid, is let in right away and has its prologue behind it when the partials arrive.
    // (With two CTAs of this grid on every SM it could only come in as they leave, and what it does then
    // slows the last of them down: measured, see the trigger below.)
    if (P.early_trigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned nseg_total = segment_count(P);

    if (threadIdx.x < 32) {
        // ---------------- producer ----------------
        if (threadIdx.x == 0) {
            unsigned st = 0, par = 1;                     // stage and the parity of its "empty" phase to wait for
            unsigned issued = 0;
            bool ok = true;
            // every CTA starts on the segment of its own number (so that a small batch spreads over all
            // CTAs however unevenly they start); the rest come from the counter
            // Half the CTAs take segments from the front of the (sequence-major) list, half from the back,
            // until the two meet.  CTAs i and i + gridDim/2 share an SM under round-robin placement, so
            // when cost varies along the batch (temperature-0 sequences stream at memory speed, the others
            // are held by the exponentials) every SM gets both kinds at once.
            const unsigned n_front = (gridDim.x + 1) / 2, n_back = gridDim.x - n_front;
            const bool back = blockIdx.x >= n_front;
            const unsigned long long one = back ? (1ull << 32) : 1ull;
            auto take = [&]() -> unsigned {               // the next segment number for this CTA, or nseg_total when none is left
                const unsigned long long old = atomicAdd(P.seg_counter, one);
                const unsigned long long f = n_front + (old & 0xffffffffull), k = n_back + (old >> 32);
                if (f + k >= nseg_total) return nseg_total;
                return back ? nseg_total - 1u - static_cast<unsigned>(k) : static_cast<unsigned>(f);
            };
            unsigned id = back ? nseg_total - 1u - (blockIdx.x - n_front) : blockIdx.x;
            Segment g = decode_segment(P, id);
            while (ok) {
                if (id >= nseg_total) break;
                finish_segment(P, g);
                const Segment gc = g;
                if (gc.skip) { id = take(); if (id < nseg_total) g = decode_segment(P, id); continue; }
                const RowView<DT> rv = segment_row<DT>(P, gc);
                const int v_end = min(gc.v1, rv.nvec());
                int v0 = gc.v0;
                do {                                     // an empty segment still sends one (empty) stage
                    const int nv = max(0, min(CVEC, v_end - v0));
                    ok = mbar_wait(&sm.empty[st], par, &sm.error, P.error);
                    if (!ok) break;
                    int f0, f1;
                    full_vectors<DT>(rv, v0, v0 + nv, f0, f1);
                    const bool interior = (f0 == v0 && f1 == v0 + nv);
                    StatsMeta mt;
                    mt.v0 = v0; mt.nv = nv;
                    mt.flags = (v0 == gc.v0 ? META_FIRST : 0) | (v0 + CVEC >= v_end ? META_LAST : 0) |
                               (interior ? META_INTERIOR : 0);
                    mt.b = gc.b; mt.row = gc.row; mt.seg = gc.seg; mt.tau = gc.tau; mt.pad = 0;
                    sm.meta[st] = mt;
                    const unsigned bytes = static_cast<unsigned>(f1 - f0) * 16u;
                    mbar_arrive_expect_tx(&sm.full[st], bytes);
                    if (bytes)
                        bulk_load(stage_base + static_cast<size_t>(st) * CVEC + (f0 - v0), rv.vec0 + f0, bytes, &sm.full[st]);
                    ++issued;
                    if (++st == NST) { st = 0; par ^= 1u; }
                    v0 += CVEC;
                } while (v0 < v_end);
                id = take();
                if (id < nseg_total) g = decode_segment(P, id);
            }
            // nothing more to start: the next kernel of the stream may be made resident as CTAs of this
            // one leave (it still waits for all of this grid before it reads the partials).  Triggering
            // earlier, when the queue runs dry, was measured: the early residents slow the last segments
            // down by as much as their prologue saves.
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            if (ok) {                                    // tell the consumers there is nothing more
                if (mbar_wait(&sm.empty[st], par, &sm.error, P.error)) {
                    StatsMeta mt;
                    mt.v0 = 0; mt.nv = 0; mt.flags = META_END; mt.b = 0; mt.row = 0; mt.seg = 0; mt.tau = 1.f; mt.pad = 0;
                    sm.meta[st] = mt;
                    mbar_arrive(&sm.full[st]);
                }
            }
            // After a timeout nobody may be waiting for the copies still in flight: let them land
            // (bounded) before this CTA's shared memory goes away.
            if (*reinterpret_cast<volatile int *>(&sm.error)) {
                const unsigned n = issued < static_cast<unsigned>(NST) ? issued : static_cast<unsigned>(NST);
                for (unsigned j = 0; j < n; ++j) {
                    const unsigned sidx = (st + NST - 1 - j) % NST;           // the last n stages issued
                    const unsigned use = (issued - 1 - j) / NST;               // how often that stage had been used before
                    for (unsigned i = 0; i < kWaitLimit && !mbar_test(&sm.full[sidx], use & 1u); ++i) __nanosleep(64);
                }
            }
        }
    } else {
        // ---------------- consumers ----------------
        const int tid = threadIdx.x - 32, lane = tid & 31, warp = tid >> 5;
        Segment g;
        g.b = 0; g.row = 0; g.v0 = g.v1 = 0; g.seg = 0; g.skip = false; g.tau = 1.f; g.m = 0;
        RowView<DT> rv(P.zt, 0, P.V_t);
        bool greedy = false, masked = false;
        float s = 0.f;
        float c_run = kNegBig, acc = 0.f;                  // softmax rows: reference, sum
        float best = -INFINITY; int best_idx = INT_MAX;    // temperature-0 rows: max, lowest index
        uint32_t best_mm = Elt<TLI_BF16>::kNegInfWord;     // ... and the packed maxima of bf16 rows
        bool clean_exit = false;
        unsigned slot = 0;                                 // where this segment's per-warp results meet
        unsigned st = 0, par = 0;                          // stage and the parity of its "full" phase to wait for
        for (;;) {
            if (!mbar_wait(&sm.full[st], par, &sm.error, P.error)) break;
            const StatsMeta meta = sm.meta[st];
            const uint4 *stage = stage_base + static_cast<size_t>(st) * CVEC;
            uint64_t *empty_bar = &sm.empty[st];
            if (++st == NST) { st = 0; par ^= 1u; }
            if (meta.flags & META_END) { clean_exit = true; break; }
            if (meta.flags & META_FIRST) {
                g.b = meta.b; g.row = meta.row; g.seg = meta.seg; g.tau = meta.tau;
                rv = segment_row<DT>(P, g);
                greedy = (g.tau == 0.f);
                masked = g.row > P.K;
                s = 1.4426950408889634f / g.tau;
                c_run = kNegBig; acc = 0.f; best = -INFINITY; best_idx = INT_MAX; best_mm = Elt<TLI_BF16>::kNegInfWord;
            }
            const int v0 = meta.v0, nv = meta.nv;
            const int nq = (nv + kSThreads - 1) / kSThreads;                  // the same for the whole CTA
            uint32_t bits[CV] = {};
            if (masked) {                                  // the mask words travel while the stage is read
#pragma unroll
                for (int q = 0; q < CV; ++q) {
                    const int i = q * kSThreads + tid;
                    bits[q] = (i < nv) ? mask_bits(P.maskbits, rv.first_elem(v0 + i) + P.d_begin) : 0u;
                }
            }
            uint4 raw[CV];
            load_stage<DT, CV>(rv, v0, nv, (meta.flags & META_INTERIOR) != 0, stage, tid, raw);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);                            // stage may be refilled now
            if (masked && !greedy) {
                if constexpr (DT == TLI_BF16) {                   // mask the packed words, then as a target row
#pragma unroll
                    for (int q = 0; q < CV; ++q) mask_bf16_vector(raw[q], bits[q]);
                }
            }
            constexpr bool kMaskInSum = (DT != TLI_BF16);          // fp32 drafter rows apply the mask element by element
            if (nq == CV) {
                if (greedy) argmax_chunk<DT, CV, true>(raw, nq, (meta.flags & META_FIRST) != 0, rv, v0 + tid, best_mm, best, best_idx);
                else if (masked && kMaskInSum) softmax_chunk<DT, CV, true, true>(raw, bits, nq, s, c_run, acc);
                else softmax_chunk<DT, CV, false, true>(raw, bits, nq, s, c_run, acc);
            } else if (nq > 0) {
                if (greedy) argmax_chunk<DT, CV, false>(raw, nq, (meta.flags & META_FIRST) != 0, rv, v0 + tid, best_mm, best, best_idx);
                else if (masked && kMaskInSum) softmax_chunk<DT, CV, true, false>(raw, bits, nq, s, c_run, acc);
                else softmax_chunk<DT, CV, false, false>(raw, bits, nq, s, c_run, acc);
            }
            if (!(meta.flags & META_LAST)) continue;

            // ---- segment done: one (reference, sum) or (max, index) pair per warp, then per CTA ----
            float px, py;
            if (greedy) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    float b2 = __shfl_xor_sync(0xffffffffu, best, o);
                    int i2 = __shfl_xor_sync(0xffffffffu, best_idx, o);
                    if (b2 > best || (b2 == best && i2 < best_idx)) { best = b2; best_idx = i2; }
                }
                px = best; py = __int_as_float(best_idx == INT_MAX ? INT_MAX : best_idx + P.t_begin);     // global id
            } else {
                // common reference first, then one exact rescale per lane and a plain sum
                const float c_w = warp_max(c_run);
                float a_w = acc * pow2_neg(c_run - c_w);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) a_w += __shfl_xor_sync(0xffffffffu, a_w, o);
                px = c_w; py = a_w;
            }
            // the last warp to arrive combines the sixteen results, always in warp order
            float2 *pairs = sm.pairs[slot];
            unsigned *arrived = &sm.arrived[slot];
            if (++slot == kPairSlots) slot = 0;
            unsigned ticket = 0;
            if (lane == 0) {
                pairs[warp] = make_float2(px, py);
                __threadfence_block();
                ticket = atomicAdd(arrived, 1u);
            }
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            if (ticket == kSWarps - 1) {
                if (lane == 0) *arrived = 0u;
                __threadfence_block();
                float2 pr;
                if (greedy) {
                    pr = (lane < kSWarps) ? ld_shared_pair(pairs + lane) : make_float2(-INFINITY, __int_as_float(INT_MAX));
                    float bb = pr.x; int ii = __float_as_int(pr.y);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        float b2 = __shfl_xor_sync(0xffffffffu, bb, o);
                        int i2 = __shfl_xor_sync(0xffffffffu, ii, o);
                        if (b2 > bb || (b2 == bb && i2 < ii)) { bb = b2; ii = i2; }
                    }
                    pr = make_float2(bb, __int_as_float(ii));
                } else {
                    pr = (lane < kSWarps) ? ld_shared_pair(pairs + lane) : make_float2(kNegBig, 0.f);
                    const float c_all = warp_max(pr.x);
                    float a_all = pr.y * pow2_neg(pr.x - c_all);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) a_all += __shfl_xor_sync(0xffffffffu, a_all, o);
                    pr = make_float2(c_all, a_all);
                }
                if (lane == 0) {
                    float2 *dst = (g.row <= P.K)
                        ? P.part_t + (static_cast<size_t>(g.b) * (P.K + 1) + g.row) * P.nst + g.seg
                        : P.part_d + (static_cast<size_t>(g.b) * P.K + (g.row - P.K - 1)) * P.nsd + g.seg;
                    __stcg(dst, pr);
                }
            }
        }
        // the last CTA to leave puts the segment counter back for the next call
        if (clean_exit && tid == 0) {
            __threadfence();
            const unsigned t = atomicAdd(P.cta_done, 1u);
            if (t == gridDim.x - 1) { *P.seg_counter = 0ull; *P.cta_done = 0u; __threadfence(); }
        }
    }
}

// ---------------------------------------------------------------------------
// decision: Algorithm 5's acceptance tests and count, once per sequence
// ---------------------------------------------------------------------------
//
// fp64 combination of the segment partials of every row of the sequence, Algorithm 5's
// acceptance tests (thresholds in fp64 from two gathered logits each) and count of accepted
// drafts, and what the sampling pass needs.  The gathers do not depend on the statistics, so they
// are issued before the wait for the statistics kernel and complete while the partials are being
// combined.  Run by all NT threads of a CTA; every thread returns the same `sel` and `flags`.
// `writer`: this CTA stores accepted / row_status / p_draft / q_draft (and next_token when the
// sequence is finished here: invalid temperature, temperature 0, non-finite logits).
// Returns true when the extra token is still to be drawn (sel.mode is MODE_RESIDUAL or
// MODE_TARGET_ONLY).
// POLL: the caller's grid did not wait for the statistics grid; the partials come from the context's
// buffer and each is waited for where it is read (load_partial_when_stored).
template <int DT, int NT, bool POLL = false>
__device__ __forceinline__ bool decide_sequence(const Params &P, int b, bool writer, RowSel &sel, int &flags) {
    const int tid = threadIdx.x;
    // loads that depend on nothing go out together: temperature, this thread's uniform, (below) its draft id
    const float tau = __ldg(P.tau + b);
    const float u_mine = (tid <= P.K) ? __ldg(P.u + static_cast<size_t>(b) * (P.K + 1) + tid) : 0.f;
    __shared__ float sm_c[2 * TLI_MAX_K + 1];      // reference (or max value for temperature 0)
    __shared__ double sm_s[2 * TLI_MAX_K + 1];     // sum (or arg-max index)
    __shared__ int sm_accept[TLI_MAX_K];
    __shared__ int sm_flags;
    __shared__ RowSel sm_sel;
    const int K = P.K;
    const int Kb = P.draft_len ? min(max(__ldg(P.draft_len + b), 0), K) : K;     // drafts of this sequence that count
    sel.n = 0; sel.mode = MODE_SKIP; sel.s = 0.f; sel.c_t = 0.f; sel.rs_t = 0.f; sel.c_d = 0.f; sel.rs_d = 0.f; sel.v = 0.f;
    if (!(tau >= 0.f) || isinf(tau)) {             // negative, NaN or infinite temperature
        flags = TLI_ROW_BAD_TEMPERATURE;
        if (!POLL) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (writer) {
            if (tid == 0) {
                P.accepted[b] = 0; P.next_token[b] = 0;
                if (P.status) P.status[b] = TLI_ROW_BAD_TEMPERATURE;
            }
            if (tid < K) {
                if (P.p_out) P.p_out[static_cast<size_t>(b) * K + tid] = 0.f;
                if (P.q_out) P.q_out[static_cast<size_t>(b) * K + tid] = 0.f;
            }
        }
        return false;
    }
    const bool greedy = (tau == 0.f);
    // the drafted token's two logits and its target id: loads in flight while the rows are combined
    int g_x = -1, g_t = -1, g_fl = 0;
    float g_zt = 0.f, g_zd = 0.f;
    if (tid < Kb) {
        g_x = __ldg(P.draft + static_cast<size_t>(b) * K + tid);
        if (g_x < 0 || g_x >= P.V_d) g_fl |= TLI_ROW_DRAFT_RANGE;
        else { g_t = __ldg(P.map + g_x); if (g_t < 0) g_fl |= TLI_ROW_DRAFT_UNMAPPED; }
        if (g_t >= 0 && !greedy) {
            g_zt = load_elt<DT>(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(tid) * P.t_sk + g_t);
            g_zd = load_elt<DT>(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(tid) * P.d_sk + g_x);
        }
    }
    const int nrows = greedy ? (K + 1) : (2 * K + 1);      // rows beyond the sequence's own drafts have no partials
    if (tid == K) sm_sel.v = u_mine;

    // everything below reads what the statistics kernel wrote (its partials, its time-out word)
    if (!POLL) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) {
        int fl = (P.n_mapped == 0 && !greedy) ? TLI_ROW_FALLBACK : 0;
        if (!POLL && *reinterpret_cast<volatile unsigned *>(P.error)) fl |= TLI_ROW_TIMEOUT;
        sm_flags = fl;
    }
    if (POLL) __syncthreads();                       // sm_flags is in place before a wait that expires ORs into it
    // Eight lanes per row, one pass: every lane folds its share of the row's partials into a running
    // pair (changes of reference are exact powers of two), then the eight lanes are folded together.
    // (the loop bound is the same for all lanes of a warp: lanes beyond the last row run along with
    // zero partials, because the shuffles below need the whole warp)
    for (int r0 = 0; r0 < nrows; r0 += NT / 8) {
        const int r = r0 + (tid >> 3);
        const int sub = tid & 7;
        const bool is_t = r <= K;
        const bool mine = r < nrows && (is_t ? r <= Kb : r - K - 1 < Kb);
        const int nseg = !mine ? 0 : (is_t ? P.nst : P.nsd);
        const float2 *part = is_t ? P.part_t + (static_cast<size_t>(b) * (K + 1) + r) * P.nst
                                  : P.part_d + (static_cast<size_t>(b) * K + (r - K - 1)) * P.nsd;
        if (greedy) {
            float best = -INFINITY; int idx = INT_MAX;
            for (int i = sub; i < nseg; i += 8) {
                float2 pr;
                if (!POLL) pr = __ldcg(part + i);
                else if (!load_partial_when_stored(part + i, P.error, pr)) {
                    atomicOr(&sm_flags, TLI_ROW_TIMEOUT);
                    pr = make_float2(-INFINITY, __int_as_float(INT_MAX));
                }
                int i2 = __float_as_int(pr.y);
                if (pr.x > best || (pr.x == best && i2 < idx)) { best = pr.x; idx = i2; }
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                float b2 = __shfl_xor_sync(0xffffffffu, best, o);
                int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                if (b2 > best || (b2 == best && i2 < idx)) { best = b2; idx = i2; }
            }
            if (sub == 0 && r < nrows) { sm_c[r] = best; sm_s[r] = (idx == INT_MAX) ? 0.0 : static_cast<double>(idx); }
        } else {
            float c = kNegBig;
            double sum = 0.0;
            for (int i = sub; i < nseg; i += 8) {
                float2 pr;
                if (!POLL) pr = __ldcg(part + i);
                else if (!load_partial_when_stored(part + i, P.error, pr)) {
                    atomicOr(&sm_flags, TLI_ROW_TIMEOUT);
                    pr = make_float2(kNegBig, 0.f);
                }
                const float cn = fmaxf(c, pr.x);
                sum = sum * pow2_neg_d(c - cn) + static_cast<double>(pr.y) * pow2_neg_d(pr.x - cn);
                c = cn;
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                const float c2 = __shfl_xor_sync(0xffffffffu, c, o);
                const double s2 = __shfl_xor_sync(0xffffffffu, sum, o);
                const float cn = fmaxf(c, c2);
                sum = sum * pow2_neg_d(c - cn) + s2 * pow2_neg_d(c2 - cn);
                c = cn;
            }
            if (sub == 0 && r < nrows) { sm_c[r] = c; sm_s[r] = sum; }
        }
    }
    __syncthreads();

    const float s_f = 1.4426950408889634f / tau;       // the same rounded scale the statistics used
    if (tid < Kb) {
        const int j = tid;
        int ok = 0, fl = g_fl;
        float pv = 0.f, qv = 0.f;
        const int t = g_t;
        if (greedy) {
            ok = (t >= 0 && t == static_cast<int>(sm_s[j]));
        } else {
            const double S_t = sm_s[j], S_d = sm_s[K + 1 + j];
            if (!(S_t > 0.0) || !isfinite(S_t) || !isfinite(S_d)) fl |= TLI_ROW_NONFINITE;
            else if (t >= 0) {
                const double sd = static_cast<double>(s_f);
                const double zt = static_cast<double>(g_zt);
                const double zd = static_cast<double>(g_zd);
                const double p = exp2(zt * sd - static_cast<double>(sm_c[j])) / S_t;
                const double q = (S_d > 0.0) ? exp2(zd * sd - static_cast<double>(sm_c[K + 1 + j])) / S_d : 0.0;
                double thr;
                if (q > 0.0) thr = fmin(1.0, p / q);
                else thr = (p > 0.0) ? 1.0 : 0.0;
                ok = static_cast<double>(u_mine) < thr;
                pv = static_cast<float>(p); qv = static_cast<float>(q);
            }
        }
        sm_accept[j] = ok;
        if (fl) atomicOr(&sm_flags, fl);
        if (writer) {
            if (P.p_out) P.p_out[static_cast<size_t>(b) * K + j] = pv;
            if (P.q_out) P.q_out[static_cast<size_t>(b) * K + j] = qv;
        }
    } else if (tid < K && writer) {
        if (P.p_out) P.p_out[static_cast<size_t>(b) * K + tid] = 0.f;
        if (P.q_out) P.q_out[static_cast<size_t>(b) * K + tid] = 0.f;
    }
    __syncthreads();
    if (tid == 0) {
        int n = Kb;
        for (int j = 0; j < Kb; ++j) if (!sm_accept[j]) { n = j; break; }
        int fl = sm_flags;
        // the row the extra token is drawn from must have a usable sum too
        if (!greedy) {
            const double S_n = sm_s[n];
            if (!(S_n > 0.0) || !isfinite(S_n)) fl |= TLI_ROW_NONFINITE;
        }
        RowSel rs;
        rs.n = n; rs.mode = MODE_SKIP; rs.s = s_f; rs.c_t = 0.f; rs.rs_t = 0.f; rs.c_d = 0.f; rs.rs_d = 0.f;
        rs.v = sm_sel.v;
        int token = -1;                            // -1: the sampling pass supplies it
        if (greedy) {
            token = static_cast<int>(sm_s[n]);
        } else if (fl & TLI_ROW_NONFINITE) {
            n = 0;
            token = 0;
        } else {
            rs.c_t = sm_c[n];
            rs.rs_t = static_cast<float>(1.0 / sm_s[n]);
            if (n < Kb) {
                const double S_d = sm_s[K + 1 + n];
                rs.mode = MODE_RESIDUAL;
                rs.c_d = sm_c[K + 1 + n];
                rs.rs_d = (S_d > 0.0) ? static_cast<float>(1.0 / S_d) : 0.f;
            } else {
                rs.mode = MODE_TARGET_ONLY;
            }
        }
        rs.n = n;
        if (writer) {
            P.accepted[b] = n;
            if (token >= 0) P.next_token[b] = token;
            if (P.status) P.status[b] = fl;
        }
        sm_sel = rs;
        sm_flags = fl;
    }
    __syncthreads();
    sel = sm_sel;
    flags = sm_flags;
    return sel.mode != MODE_SKIP;
}

// The decision as a kernel of its own, one CTA per sequence (the form for vocabularies too large
// for the cluster kernel below): leaves a RowSel per sequence for the tile kernel.
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_decide_kernel(const Params P) {
    RowSel sel;
    int flags;
    decide_sequence<DT, kThreads>(P, blockIdx.x, true, sel, flags);
    if (threadIdx.x == 0) P.sel[blockIdx.x] = sel;
}

// ---------------------------------------------------------------------------
// pass 2: the extra token
// ---------------------------------------------------------------------------

// Weights of the elements of vector v of the sampled target row:
// p(t), or max(0, p(t) - q'(inv[t])) for the residual.  The same code feeds the
// tile sums and every rescan, so the levels of the CDF walk agree bit for bit.
// LEAN: the caller knows that the vector lies wholly inside the row and that its first id is a
// multiple of four (true for every vector of a tile that is not at an end of an aligned row), which
// takes the checks and the element-wise loads out of the code.
template <int DT> __device__ __forceinline__ float load_elt_shared(uint32_t row_addr, int i) {
    if (DT == TLI_F32) {
        float v;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(row_addr + static_cast<uint32_t>(i) * 4u));
        return v;
    }
    unsigned short h;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(row_addr + static_cast<uint32_t>(i) * 2u));
    return __uint_as_float(static_cast<uint32_t>(h) << 16);
}

// Where the drafter logits of row n come from: the row in global memory, a copy of it staged in
// shared memory (zd_row is then its shared-memory address), or -- vocabulary-sharded calls -- the
// slices of it gathered from all shards (zd_row is then the slice of shard 0; drafter id x lies
// x / sh_wd slices further on).
enum : int { SRC_GLOBAL = 0, SRC_SHARED = 1, SRC_SHARDS = 2 };

// p(t) and q'_T(t) of the elements of one vector of the sampled target row.
// LEAN: the caller knows that the vector lies wholly inside the row and that the global id of its
// first element is a multiple of four, which takes the checks and the element-wise loads out.
template <int DT, bool LEAN, int SRC>
__device__ __forceinline__ void vector_p_q(const Params &P, const RowSel &sel, const uint4 &raw, int e0,
                                           const void *zd_row, float (&pt)[Elt<DT>::kPerVec], float (&q)[Elt<DT>::kPerVec]) {
    constexpr int EPV = Elt<DT>::kPerVec;
    float z[EPV];
    unpack<DT>(raw, z);
    int x[EPV];
#pragma unroll
    for (int i = 0; i < EPV; ++i) x[i] = -1;
    if (sel.mode == MODE_RESIDUAL) {
        const int g0 = e0 + P.t_begin;                         // global target id of the vector's first element
        if (LEAN || (e0 >= 0 && e0 + EPV <= P.V_t && (g0 & 3) == 0)) {
#pragma unroll
            for (int i = 0; i < EPV; i += 4) {
                const int4 u = __ldg(reinterpret_cast<const int4 *>(P.inv + g0 + i));
                x[i] = u.x; x[i + 1] = u.y; x[i + 2] = u.z; x[i + 3] = u.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                const int t = e0 + i;
                x[i] = (t >= 0 && t < P.V_t) ? __ldg(P.inv + g0 + i) : -1;
            }
        }
    }
    const float nct = -sel.c_t, ncd = -sel.c_d;
#pragma unroll
    for (int i = 0; i < EPV; ++i) {
        pt[i] = __fmul_rn(ex2(__fmaf_rn(z[i], sel.s, nct)), sel.rs_t);
        q[i] = 0.f;
        if (x[i] >= 0) {
            float zdv;
            if (SRC == SRC_SHARED) {
                zdv = load_elt_shared<DT>(static_cast<uint32_t>(reinterpret_cast<uintptr_t>(zd_row)), x[i]);
            } else if (SRC == SRC_SHARDS) {
                const int g = x[i] / P.sh_wd;
                zdv = load_elt<DT>(zd_row, static_cast<long long>(g) * P.sh_stride + (x[i] - g * P.sh_wd));
            } else {
                zdv = load_elt<DT>(zd_row, x[i]);
            }
            q[i] = __fmul_rn(ex2(__fmaf_rn(zdv, sel.s, ncd)), sel.rs_d);
        }
    }
}

template <int DT, bool LEAN = false, int SRC = SRC_GLOBAL>
__device__ __forceinline__ void vector_weights_from(const Params &P, const RowSel &sel, const uint4 &raw, int e0,
                                                    const void *zd_row, float (&w)[Elt<DT>::kPerVec]) {
    constexpr int EPV = Elt<DT>::kPerVec;
    float pt[EPV], q[EPV];
    vector_p_q<DT, LEAN, SRC>(P, sel, raw, e0, zd_row, pt, q);
    // p and q' are each rounded before the subtraction, so that equal distributions leave exactly 0
#pragma unroll
    for (int i = 0; i < EPV; ++i) w[i] = fmaxf(0.f, __fsub_rn(pt[i], q[i]));
}

template <int DT, bool LEAN = false, int SRC = SRC_GLOBAL>
__device__ __forceinline__ void vector_weights(const Params &P, const RowSel &sel, const RowView<DT> &rt,
                                               const void *zd_row, int v, float (&w)[Elt<DT>::kPerVec]) {
    const uint4 raw = LEAN ? __ldg(rt.vec0 + v) : rt.load(v);
    vector_weights_from<DT, LEAN, SRC>(P, sel, raw, rt.first_elem(v), zd_row, w);
}

template <int N> __device__ __forceinline__ float ordered_sum(const float (&w)[N]) {
    float s = w[0];
#pragma unroll
    for (int i = 1; i < N; ++i) s = __fadd_rn(s, w[i]);
    return s;
}

// sum of one tile's weights (fp64 over fp32 vector sums); result valid in thread 0
template <int DT>
__device__ __forceinline__ double tile_weight_sum(const Params &P, const RowSel &sel, const RowView<DT> &rt,
                                                  const void *zd_row, int tile, double *sm_red) {
    constexpr int EPV = Elt<DT>::kPerVec;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = rt.nvec();
    double acc = 0.0;
    const int v_first = tile * kVecPerTile;
    const bool lean = (rt.head & 3) == 0 && (P.t_begin & 3) == 0 && rt.first_elem(v_first) >= 0 &&
                      rt.first_elem(v_first + kVecPerTile - 1) + EPV <= rt.V;        // the same for the whole CTA
    if (lean) {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            float w[EPV];
            vector_weights<DT, true>(P, sel, rt, zd_row, v_first + k * kThreads + tid, w);
            acc += static_cast<double>(ordered_sum(w));
        }
    } else {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int v = v_first + k * kThreads + tid;
            if (v < nvec) {
                float w[EPV];
                vector_weights<DT>(P, sel, rt, zd_row, v, w);
                acc += static_cast<double>(ordered_sum(w));
            }
        }
    }
    acc = warp_sum(acc);
    __syncthreads();                   // sm_red may still be in use by the previous tile
    if (lane == 0) sm_red[warp] = acc;
    __syncthreads();
    double tot = 0.0;
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < kWarps; ++i) tot += sm_red[i];
    }
    return tot;
}

// The last two levels of the CDF inversion by one CTA: the vector of tile T that holds `rem` (the
// part of v * total that falls into the tile), then the element of that vector.
// KEEP: each thread forms the weights of four consecutive vectors of the tile and keeps them in
// registers, so that the final walk needs no second trip to memory (kernels that have the
// registers); otherwise the vector the target falls into is formed again (inside the sampling
// kernel, whose 32 registers per thread would spill them).
template <int DT, bool KEEP, int SRC>
__device__ void walk_tile(const Params &P, int b, const RowSel &sel, const RowView<DT> &rt, const void *zd_row,
                          int T, double rem) {
    constexpr int EPV = Elt<DT>::kPerVec;
    __shared__ float sm_seg[kVecPerTile];
    __shared__ double sm_warp_tot[kWarps];
    __shared__ int sm_found, sm_lastpos;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = rt.nvec();
    // vector sums of tile T; thread i owns vectors 4i .. 4i+3 in the block-wide exclusive prefix (fp64)
    float wv[KEEP ? kVecPerThread : 1][EPV];
    double loc[kVecPerThread];
    double mine = 0.0;
    if constexpr (KEEP) {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int v = T * kVecPerTile + tid * kVecPerThread + k;
            float sseg = 0.f;
            if (v < nvec) {
                vector_weights<DT, false, SRC>(P, sel, rt, zd_row, v, wv[k]);
                sseg = ordered_sum(wv[k]);
            } else {
#pragma unroll
                for (int i = 0; i < EPV; ++i) wv[k][i] = 0.f;
            }
            loc[k] = static_cast<double>(sseg); mine += loc[k];
        }
        if (tid == 0) { sm_found = INT_MAX; sm_lastpos = -1; }
    } else {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int g = k * kThreads + tid;
            const int v = T * kVecPerTile + g;
            float sseg = 0.f;
            if (v < nvec) {
                float w[EPV];
                vector_weights<DT, false, SRC>(P, sel, rt, zd_row, v, w);
                sseg = ordered_sum(w);
            }
            sm_seg[g] = sseg;
        }
        if (tid == 0) { sm_found = INT_MAX; sm_lastpos = -1; }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) { loc[k] = static_cast<double>(sm_seg[tid * kVecPerThread + k]); mine += loc[k]; }
    }
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) sm_warp_tot[warp] = incl;
    __syncthreads();
    double base = 0.0;
    for (int i = 0; i < warp; ++i) base += sm_warp_tot[i];
    double run = base + incl - mine;               // mass before this thread's first vector
    int cand = INT_MAX, lastpos = -1;
    double cand_before = 0.0;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const double nx = run + loc[k];
        if (loc[k] > 0.0) lastpos = tid * kVecPerThread + k;
        if (cand == INT_MAX && nx > rem) { cand = tid * kVecPerThread + k; cand_before = run; }
        run = nx;
    }
    if (cand != INT_MAX) atomicMin(&sm_found, cand);
    if (lastpos >= 0) atomicMax(&sm_lastpos, lastpos);
    __syncthreads();
    const int found = sm_found;
    const int G = (found != INT_MAX) ? found : sm_lastpos;
    if (G < 0) {                                   // cannot happen when the tile has positive mass
        if (tid == 0) P.next_token[b] = 0;
        return;
    }
    if (tid == G / kVecPerThread) {
        // walk the elements of vector G with the same running fp32 sum that formed its total;
        // when rounding left no vector above the target, take the last positive element instead
        double before = 0.0;
        if (found != INT_MAX) {
            before = base + incl - mine;
            for (int k = 0; k < G - tid * kVecPerThread; ++k) before += loc[k];
        }
        const double rem2 = (found != INT_MAX) ? (rem - before) : INFINITY;
        float w[EPV];
        const int v = T * kVecPerTile + G;
        if constexpr (KEEP) {
#pragma unroll
            for (int k = 0; k < kVecPerThread; ++k)
                if (k == G - tid * kVecPerThread) {
#pragma unroll
                    for (int i = 0; i < EPV; ++i) w[i] = wv[k][i];
                }
        } else {
            vector_weights<DT, false, SRC>(P, sel, rt, zd_row, v, w);
        }
        float runf = 0.f;
        int pick = -1, lastw = 0;
#pragma unroll
        for (int i = 0; i < EPV; ++i) {
            runf = (i == 0) ? w[0] : __fadd_rn(runf, w[i]);
            if (w[i] > 0.f) lastw = i;
            if (pick < 0 && static_cast<double>(runf) > rem2) pick = i;
        }
        if (pick < 0) pick = lastw;
        int token = rt.first_elem(v) + pick;
        token = min(max(token, 0), P.V_t - 1);
        P.next_token[b] = token + P.t_begin;
    }
}

// The CDF inversion for one sequence by one CTA, tile -> vector -> element, from the tile sums in
// the workspace.  Either the last CTA of the sampling kernel to finish a tile of the sequence runs
// it, or (large batches) the selection kernel does, one CTA per sequence.
template <int DT, bool KEEP = false>
__device__ void select_sequence(const Params &P, int b, RowSel sel, const RowView<DT> &rt, const void *zd_row) {
    __shared__ double sm_red[kWarps];
    __shared__ double sm_tiles[kMaxTiles];
    __shared__ int sm_tile, sm_retry;
    __shared__ double sm_rem;
    const int tid = threadIdx.x;
    const int ntile = P.ntile;
    // ---- last CTA of the sequence: invert the CDF, tile -> vector -> element ----
    for (int i = tid; i < ntile; i += kThreads) sm_tiles[i] = __ldcg(P.tilesum + static_cast<size_t>(b) * ntile + i);
    __syncthreads();
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (tid == 0) {
            double R = 0.0;
            for (int i = 0; i < ntile; ++i) R += sm_tiles[i];
            sm_retry = 0;
            if (!(R > 0.0) || !isfinite(R)) {
                sm_retry = 1;
            } else {
                const double target = static_cast<double>(sel.v) * R;
                double run = 0.0;
                int T = -1, lastpos = 0;
                double before = 0.0;
                for (int i = 0; i < ntile; ++i) {
                    const double nx = run + sm_tiles[i];
                    if (sm_tiles[i] > 0.0) lastpos = i;
                    if (T < 0 && nx > target) { T = i; before = run; }
                    run = nx;
                }
                if (T < 0) { T = lastpos; before = R - sm_tiles[lastpos]; }
                sm_tile = T;
                sm_rem = target - before;
            }
        }
        __syncthreads();
        if (!sm_retry) break;
        if (attempt == 1) {                      // no usable mass even from p: give up on the row
            if (tid == 0) {
                P.next_token[b] = 0;
                if (P.status) P.status[b] |= TLI_ROW_NONFINITE;
            }
            return;
        }
        // zero residual mass: sample from p of the same position instead
        sel.mode = MODE_TARGET_ONLY;
        if (tid == 0 && P.status) P.status[b] |= TLI_ROW_FALLBACK;
        for (int i = 0; i < ntile; ++i) {
            const double t2 = tile_weight_sum<DT>(P, sel, rt, zd_row, i, sm_red);
            if (tid == 0) sm_tiles[i] = t2;
        }
        __syncthreads();
    }

    walk_tile<DT, KEEP, SRC_GLOBAL>(P, b, sel, rt, zd_row, sm_tile, sm_rem);
}

// The sampling pass: one CTA per 16 KB tile of the target row the extra token is drawn from
// (blockIdx.y = sequence).  With P.split_select the kernel only leaves the tile sums; otherwise
// the last CTA of a sequence (atomic ticket, nobody waits) goes on to invert the CDF.
template <int DT>
__global__ void __launch_bounds__(kThreads, 8) tli_sample_kernel(const Params P) {
    __shared__ double sm_red[kWarps];
    __shared__ int sm_last;
    const int b = blockIdx.y, tile = blockIdx.x;
    const int tid = threadIdx.x;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the selection kernel, or the next call's first kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const RowSel sel = P.sel[b];
    if (sel.mode == MODE_SKIP) return;
    const int ntile = P.ntile;
    RowView<DT> rt(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(sel.n) * P.t_sk, P.V_t);
    const void *zd_row = reinterpret_cast<const char *>(P.zd) +
        (static_cast<long long>(b) * P.d_sb + static_cast<long long>(sel.n < P.K ? sel.n : 0) * P.d_sk) * Elt<DT>::kBytes;

    const double tot = tile_weight_sum<DT>(P, sel, rt, zd_row, tile, sm_red);
    if (tid == 0) {
        __stcg(P.tilesum + static_cast<size_t>(b) * ntile + tile, tot);
        sm_last = 0;
        if (!P.split_select) {
            __threadfence();
            const unsigned ticket = atomicAdd(P.cnt_sample + b, 1u);
            sm_last = (ticket == static_cast<unsigned>(ntile) - 1);
            if (sm_last) P.cnt_sample[b] = 0;
        }
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    select_sequence<DT>(P, b, sel, rt, zd_row);
}

// Large batches: the CDF inversions as a kernel of their own, one CTA per sequence, so that the
// tile CTAs of the sampling kernel carry neither a fence nor a ticket.
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_select_kernel(const Params P) {
    const int b = blockIdx.x;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the next call's first kernel may be set up meanwhile
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const RowSel sel = P.sel[b];
    if (sel.mode == MODE_SKIP) return;
    RowView<DT> rt(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(sel.n) * P.t_sk, P.V_t);
    const void *zd_row = reinterpret_cast<const char *>(P.zd) +
        (static_cast<long long>(b) * P.d_sb + static_cast<long long>(sel.n < P.K ? sel.n : 0) * P.d_sk) * Elt<DT>::kBytes;
    select_sequence<DT, true>(P, b, sel, rt, zd_row);
}

// ---------------------------------------------------------------------------
// decision and extra token in one launch: one thread-block cluster per sequence
// ---------------------------------------------------------------------------
//
// The form for vocabularies whose drafter row fits one CTA's shared memory (every bf16 vocabulary
// of today's models) and for moderate batches.  Each CTA of the cluster repeats the (cheap)
// decision, then owns one slice of target row n:
//   staging   one bulk copy brings drafter row n into the CTA's shared memory while the first
//             loads of the target slice and of the inverse map are already on their way: the
//             gather q'(inv[t]) then costs a shared-memory access instead of a second trip to L2;
//   weights   max(0, p - q'_T) (or p) per element with vector_weights_from, one fp32 sum per
//             16-byte vector kept in shared memory;
//   inversion block-wide fp64 prefix over the vector sums, the CTA totals exchanged through
//             distributed shared memory, and the CTA holding v * total walks vector -> element.
// Two cluster barriers and two trips to memory after the statistics are in, against three kernel
// boundaries and about ten dependent trips of the tile form.  Every CTA of a cluster takes the
// same branches (they decide from the same data), so the barriers always meet.

constexpr int kFinThreads = 512;                   // 1024 threads where one CTA has an SM to itself: measured slower (64 registers)
constexpr int kFinWarps = kFinThreads / 32;
constexpr int kFinMaxCluster = 16;                 // beyond 8 CTAs a cluster is not portable: the context asks the driver once

__device__ __forceinline__ unsigned cluster_cta_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned cluster_cta_count() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, unsigned rank) {      // the same offset in CTA `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f64(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}

template <int DT>
__device__ __forceinline__ void finish_sequence(const Params &P) {
    constexpr int EPV = Elt<DT>::kPerVec;
    extern __shared__ __align__(16) unsigned char fin_smem[];
    __shared__ double sm_warp_tot[kFinWarps];
    __shared__ double sm_cta_tot[2][kFinMaxCluster];       // one set per attempt
    __shared__ int sm_found, sm_lastpos, sm_error;
    __shared__ uint64_t sm_bar;
    const int b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned rank = cluster_cta_rank(), C = cluster_cta_count();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the next call's first kernel may be set up meanwhile
    const int slice = P.fin_slice;                           // vectors of the target row per CTA
    uint4 *drow = reinterpret_cast<uint4 *>(fin_smem);       // drafter row n on its 16-byte vector grid
    float *vsum = reinterpret_cast<float *>(fin_smem + static_cast<size_t>(P.fin_dvec) * 16);

    if (tid == 0) {
        mbar_init(&sm_bar, 1);
        sm_error = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    RowSel sel;
    int flags;
    bool draw;
    if (P.poll_parts) {
        // The partials lie in the context's own buffer and are waited for one by one: this grid does not
        // wait for the statistics grid as a whole (whose end reaches a waiting grid only 2.5 us after its
        // last CTA has left).  When every CTA of the cluster has read them, the first one puts the
        // slots back to "empty" for the next call.
        draw = decide_sequence<DT, kFinThreads, true>(P, b, rank == 0, sel, flags);
        cluster_barrier();        // ... and every CTA of the cluster is running before anybody stores into a neighbour
        if (rank == 0) {
            const float tau = __ldg(P.tau + b);
            if (tau >= 0.f && !isinf(tau)) {
                const int Kb = P.draft_len ? min(max(__ldg(P.draft_len + b), 0), P.K) : P.K;
                const int n_t = (Kb + 1) * P.nst, n_d = (tau == 0.f) ? 0 : Kb * P.nsd;
                float2 *pt = P.part_t + static_cast<size_t>(b) * (P.K + 1) * P.nst;
                float2 *pd = P.part_d + static_cast<size_t>(b) * P.K * P.nsd;
                const float2 empty = make_float2(__uint_as_float(kPartEmpty), __uint_as_float(kPartEmpty));
                for (int i = tid; i < n_t; i += kFinThreads) __stcg(pt + i, empty);
                for (int i = tid; i < n_d; i += kFinThreads) __stcg(pd + i, empty);
            }
        }
    } else {
        cluster_barrier();        // every CTA of the cluster is running before anybody stores into a neighbour
        draw = decide_sequence<DT, kFinThreads>(P, b, rank == 0, sel, flags);
    }
    if (!draw) return;

    const RowView<DT> rt(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(sel.n) * P.t_sk, P.V_t);
    const int nvec = rt.nvec();
    const int v_begin = static_cast<int>(rank) * slice;
    const int count = max(0, min(slice, nvec - v_begin));    // this CTA's vectors: v_begin .. v_begin + count
    uint32_t zd_smem = 0;                                    // shared-memory address of element 0 of the staged row

    if (sel.mode == MODE_RESIDUAL && count > 0) {
        const RowView<DT> rd(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(sel.n) * P.d_sk, P.V_d);
        int v0, v1;
        full_vectors<DT>(rd, 0, rd.nvec(), v0, v1);            // the vectors wholly inside the row: [v0, v1)
        if (tid == 0) {
            const unsigned bytes = static_cast<unsigned>(v1 - v0) * 16u;
            mbar_arrive_expect_tx(&sm_bar, bytes);
            if (bytes) bulk_load(drow + v0, rd.vec0 + v0, bytes, &sm_bar);
        }
        // the at most two ragged vectors of the row, element by element
        const int nvec_d = rd.nvec();
        if (tid == 32 && v0 > 0) drow[0] = rd.load(0);
        if (tid == 64 && v1 < nvec_d) drow[nvec_d - 1] = rd.load(nvec_d - 1);
        zd_smem = smem_addr(drow) + static_cast<uint32_t>(rd.head) * Elt<DT>::kBytes;
    }
    // the first vectors of the slice and their inverse-map entries travel while the row is staged
    const bool lean = (rt.head & 3) == 0 && count > 0 && rt.first_elem(v_begin) >= 0 &&
                      rt.first_elem(v_begin + count - 1) + EPV <= rt.V;                  // the same for the whole CTA
    if (sel.mode == MODE_RESIDUAL && count > 0) {
        mbar_wait(&sm_bar, 0u, &sm_error, P.error);
        __syncthreads();                                     // the ragged vectors too
    }

    const double v_target = static_cast<double>(sel.v);
    const void *zd_arg = reinterpret_cast<const void *>(static_cast<uintptr_t>(zd_smem));
    for (int attempt = 0; attempt < 2; ++attempt) {
        // ---- weights of this CTA's slice, one fp32 sum per vector ----
        if (lean) {
#pragma unroll 2
            for (int i = tid; i < count; i += kFinThreads) {
                float w[EPV];
                vector_weights<DT, true, SRC_SHARED>(P, sel, rt, zd_arg, v_begin + i, w);
                vsum[i] = ordered_sum(w);
            }
        } else {
            for (int i = tid; i < count; i += kFinThreads) {
                float w[EPV];
                vector_weights<DT, false, SRC_SHARED>(P, sel, rt, zd_arg, v_begin + i, w);
                vsum[i] = ordered_sum(w);
            }
        }
        __syncthreads();
        // ---- fp64 prefix: thread i owns the run of vectors [i * len, (i + 1) * len) ----
        const int len = (slice + kFinThreads - 1) / kFinThreads;
        const int r0 = min(tid * len, count), r1 = min(r0 + len, count);
        double mine = 0.0;
        for (int i = r0; i < r1; ++i) mine += static_cast<double>(vsum[i]);
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sm_warp_tot[warp] = incl;
        if (tid == 0) { sm_found = INT_MAX; sm_lastpos = -1; }
        __syncthreads();
        double base = 0.0, cta_total = 0.0;
#pragma unroll
        for (int i = 0; i < kFinWarps; ++i) {
            if (i == warp) base = cta_total;
            cta_total += sm_warp_tot[i];
        }
        if (tid < static_cast<int>(C))                       // this CTA's total to every CTA of the cluster
            st_cluster_f64(cluster_addr(smem_addr(&sm_cta_tot[attempt][rank]), static_cast<unsigned>(tid)), cta_total);
        cluster_barrier();
        // ---- which CTA holds v * R (the same arithmetic in every CTA) ----
        double R = 0.0;
        for (unsigned r = 0; r < C; ++r) R += sm_cta_tot[attempt][r];
        if (!(R > 0.0) || !isfinite(R)) {
            if (attempt == 1 || sel.mode == MODE_TARGET_ONLY) {          // no usable mass even from p: give up on the row
                if (rank == 0 && tid == 0) {
                    P.next_token[b] = 0;
                    if (P.status) P.status[b] = flags | TLI_ROW_NONFINITE;
                }
                return;
            }
            // zero residual mass: sample from p of the same position instead
            sel.mode = MODE_TARGET_ONLY;
            flags |= TLI_ROW_FALLBACK;
            if (rank == 0 && tid == 0 && P.status) P.status[b] = flags;
            continue;
        }
        const double target = v_target * R;
        int owner = -1, lastpos_cta = 0;
        double before = 0.0, run_c = 0.0;
        for (unsigned r = 0; r < C; ++r) {
            const double tr = sm_cta_tot[attempt][r];
            const double nx = run_c + tr;
            if (tr > 0.0) lastpos_cta = static_cast<int>(r);
            if (owner < 0 && nx > target) { owner = static_cast<int>(r); before = run_c; }
            run_c = nx;
        }
        if (owner < 0) { owner = lastpos_cta; before = R - sm_cta_tot[attempt][lastpos_cta]; }
        if (static_cast<int>(rank) != owner) return;
        // ---- this CTA: vector, then element ----
        if (sm_error && tid == 0 && P.status) P.status[b] = flags | TLI_ROW_TIMEOUT;      // the staging wait ran out
        const double rem = target - before;
        double run = base + incl - mine;                 // mass before this thread's first vector
        int cand = INT_MAX, lastpos = -1;
        double cand_before = 0.0;
        for (int i = r0; i < r1; ++i) {
            const double wv = static_cast<double>(vsum[i]);
            const double nx = run + wv;
            if (wv > 0.0) lastpos = i;
            if (cand == INT_MAX && nx > rem) { cand = i; cand_before = run; }
            run = nx;
        }
        if (cand != INT_MAX) atomicMin(&sm_found, cand);
        if (lastpos >= 0) atomicMax(&sm_lastpos, lastpos);
        __syncthreads();
        const int found = sm_found;
        const int G = (found != INT_MAX) ? found : sm_lastpos;
        if (G < 0) {                                     // cannot happen when the slice has positive mass
            if (tid == 0) P.next_token[b] = 0;
            return;
        }
        if ((found != INT_MAX) ? (cand == found) : (tid == 0)) {
            // walk the elements of vector G with the same running fp32 sum that formed its total;
            // when rounding left no vector above the target, take the last positive element instead
            const double rem2 = (found != INT_MAX) ? (rem - cand_before) : INFINITY;
            float w[EPV];
            if (lean) vector_weights<DT, true, SRC_SHARED>(P, sel, rt, zd_arg, v_begin + G, w);
            else vector_weights<DT, false, SRC_SHARED>(P, sel, rt, zd_arg, v_begin + G, w);
            float runf = 0.f;
            int pick = -1, lastw = 0;
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                runf = (i == 0) ? w[0] : __fadd_rn(runf, w[i]);
                if (w[i] > 0.f) lastw = i;
                if (pick < 0 && static_cast<double>(runf) > rem2) pick = i;
            }
            if (pick < 0) pick = lastw;
            int token = rt.first_elem(v_begin + G) + pick;
            token = min(max(token, 0), P.V_t - 1);
            P.next_token[b] = token;
        }
        return;
    }
}

template <int DT>
__global__ void __launch_bounds__(kFinThreads, 2) tli_finish_kernel(const Params P) {
    finish_sequence<DT>(P);
    if (P.poll_parts) {
        // This grid did not wait for the statistics grid; it must not be over before that grid is (whose
        // last CTA puts the segment counter back), or the kernel after this one could overtake it.  By
        // now the wait returns at once.  A time-out anywhere in that grid marks the row as it always did.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (threadIdx.x == 0 && cluster_cta_rank() == 0 && P.status && *reinterpret_cast<volatile unsigned *>(P.error))
            P.status[blockIdx.y] |= TLI_ROW_TIMEOUT;
    }
}

// ---------------------------------------------------------------------------
// drafting: one id per drafter row from q' (Algorithm 4 as a sampling distribution)
// ---------------------------------------------------------------------------
//
// One pass over the logits.  A CTA takes a 16 KB tile of a drafter row, each of its warps a 2 KB
// strip of it (128 vectors, vector k*32 + lane to lane `lane`), and nothing in a strip needs
// another warp: the strip leaves (c, S), its own integer-valued reference c = ceil(max * s) over
// the ids inside the intersection and S = sum 2^(z*s - c) over them, fp32 per vector and fp64
// across vectors.  Then one CTA per row -- the last tile CTA to finish (atomic ticket, nobody
// waits) or, for large batches, a second kernel -- brings the strips to the row's reference by
// exact powers of two, finds the strip the target v * total falls into, and one warp walks that
// strip vector by vector and element by element with sums formed by the code that formed S.

constexpr int kStripsPerTile = kWarps;
constexpr int kMaxStrips = kMaxTiles * kStripsPerTile;

struct __align__(16) DraftPart {
    double S;      // weight of the strip at its own reference (temperature 0: the strip's best id)
    float c;       // the strip's reference (temperature 0: the strip's largest logit)
    int flags;     // temperature 0: TLI_ROW_NONFINITE if an id inside the intersection holds NaN or +inf
};
struct DraftParams {
    int B, R, V_d, ntile, nstrip, split;     // V_d: length of a row (the target vocabulary when no mask is given)
    const void *zd; long long d_sb, d_sr;
    const uint32_t *maskbits;                // ids that can be drawn; NULL: every id of the row
    const int *lengths;                      // NULL, or per sequence the last row to sample (rows beyond it get -1)
    const float *tau; const float *u;
    int *draft_ids; float *q_out; int *status;
    DraftPart *part;               // [B*R][nstrip]
    unsigned *cnt;                 // [B*R] tickets, zero between calls
};

// Vector v of a drafter row with the ids outside the intersection (and outside the row) set to -inf.
// INTERIOR: the caller knows that the vector lies wholly inside the row (a whole strip does, for all
// but the two ends of a row), which takes the checks and the element-wise loads out of the code.
template <int DT, bool INTERIOR>
__device__ __forceinline__ uint4 draft_masked_vector(const DraftParams &P, const RowView<DT> &rv, int v, int nvec,
                                                     uint32_t &bits) {
    constexpr uint32_t NI = Elt<DT>::kNegInfWord;
    constexpr int EPV = Elt<DT>::kPerVec;
    bits = 0u;
    if (!INTERIOR && v >= nvec) return make_uint4(NI, NI, NI, NI);
    uint4 raw = INTERIOR ? __ldg(rv.vec0 + v) : rv.load(v);
    const int e0 = rv.first_elem(v);
    if (P.maskbits == nullptr) {                           // no mask: the elements inside the row (load() gave -inf elsewhere)
        bits = (1u << EPV) - 1u;
        if (!INTERIOR) {
            if (e0 < 0) bits &= ~((1u << (-e0)) - 1u);
            if (e0 + EPV > rv.V) bits &= (1u << (rv.V - e0)) - 1u;
        }
        return raw;
    }
    bits = mask_bits(P.maskbits, e0);
    if constexpr (DT == TLI_BF16) {
        mask_bf16_vector(raw, bits);
    } else {
        raw.x = (bits & 1u) ? raw.x : NI; raw.y = (bits & 2u) ? raw.y : NI;
        raw.z = (bits & 4u) ? raw.z : NI; raw.w = (bits & 8u) ? raw.w : NI;
    }
    return raw;
}

// This lane's kVecPerThread vectors of strip `strip` (vector k*32 + lane of the strip's 128).
template <int DT>
__device__ __forceinline__ void draft_load_strip(const DraftParams &P, const RowView<DT> &rv, int strip, int nvec, int lane,
                                                 uint4 (&m)[kVecPerThread], uint32_t (&bits)[kVecPerThread]) {
    const int v0 = strip * (32 * kVecPerThread);
    const bool interior = rv.first_elem(v0) >= 0 &&
                          rv.first_elem(v0 + 32 * kVecPerThread - 1) + Elt<DT>::kPerVec <= rv.V;
    if (interior) {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) m[k] = draft_masked_vector<DT, true>(P, rv, v0 + k * 32 + lane, nvec, bits[k]);
    } else {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) m[k] = draft_masked_vector<DT, false>(P, rv, v0 + k * 32 + lane, nvec, bits[k]);
    }
}

// fp32 sum, in element order, of the weights 2^(z*s + nc) of one masked vector; the weights in w[]
template <int DT>
__device__ __forceinline__ float draft_vector_sum(const uint4 &m, float s, float nc, float (&w)[Elt<DT>::kPerVec]) {
    float z[Elt<DT>::kPerVec];
    unpack<DT>(m, z);
#pragma unroll
    for (int i = 0; i < Elt<DT>::kPerVec; ++i) w[i] = ex2(__fmaf_rn(z[i], s, nc));
    return ordered_sum(w);
}

__device__ __forceinline__ DraftPart load_part(const DraftPart *p) {
    const double2 raw = __ldcg(reinterpret_cast<const double2 *>(p));
    return *reinterpret_cast<const DraftPart *>(&raw);
}
__device__ __forceinline__ void store_part(DraftPart *p, const DraftPart &v) {
    __stcg(reinterpret_cast<double2 *>(p), *reinterpret_cast<const double2 *>(&v));
}
__device__ __forceinline__ bool better(float b2, int i2, float best, int idx) {   // larger logit, then lower id
    return i2 != INT_MAX && (idx == INT_MAX || b2 > best || (b2 == best && i2 < idx));
}
// 2^k * x for an integer-valued k >= 0
__device__ __forceinline__ double scale_up(double x, float k) { return scalbn(x, static_cast<int>(k)); }

// The id of one row from its strips' (c, S), by one CTA.
template <int DT>
__device__ void draft_select(const DraftParams &P, int row, const RowView<DT> &rv, float tau) {
    constexpr int EPV = Elt<DT>::kPerVec;
    __shared__ double sm_S[kMaxStrips];
    __shared__ float sm_c[kMaxStrips];
    __shared__ double sm_warp_tot[kWarps];
    __shared__ float sm_wmax[kWarps];
    __shared__ int sm_widx[kWarps];
    __shared__ int sm_flag, sm_found, sm_lastpos, sm_none;
    __shared__ double sm_rem, sm_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nstrip = P.nstrip;
    const bool greedy = (tau == 0.f);
    if (tid == 0) { sm_flag = 0; sm_found = INT_MAX; sm_lastpos = -1; sm_none = 0; }
    __syncthreads();
    const int per = (nstrip + kThreads - 1) / kThreads;      // consecutive strips per thread
    const int i0 = tid * per, i1 = min(i0 + per, nstrip);
    float cmax = kNegBig; int bidx = INT_MAX; int flags = 0;
    for (int i = i0; i < i1; ++i) {
        const DraftPart pt = load_part(P.part + static_cast<size_t>(row) * nstrip + i);
        sm_S[i] = pt.S; sm_c[i] = pt.c; flags |= pt.flags;
        if (greedy) {
            const int i2 = static_cast<int>(pt.S);
            if (better(pt.c, i2, cmax, bidx)) { cmax = pt.c; bidx = i2; }
        } else {
            cmax = fmaxf(cmax, pt.c);
        }
    }
    if (flags) atomicOr(&sm_flag, flags);
    if (greedy) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float b2 = __shfl_xor_sync(0xffffffffu, cmax, o);
            const int i2 = __shfl_xor_sync(0xffffffffu, bidx, o);
            if (better(b2, i2, cmax, bidx)) { cmax = b2; bidx = i2; }
        }
        if (lane == 0) { sm_wmax[warp] = cmax; sm_widx[warp] = bidx; }
        __syncthreads();
        if (tid == 0) {
            float bb = sm_wmax[0]; int ii = sm_widx[0];
            for (int i = 1; i < kWarps; ++i) if (better(sm_wmax[i], sm_widx[i], bb, ii)) { bb = sm_wmax[i]; ii = sm_widx[i]; }
            int status = sm_flag, d = ii;
            if (status & TLI_ROW_NONFINITE) d = -1;
            else if (ii == INT_MAX) { d = -1; status |= TLI_ROW_FALLBACK; }
            P.draft_ids[row] = d;
            if (P.q_out) P.q_out[row] = d >= 0 ? 1.f : 0.f;
            if (P.status) P.status[row] = status;
        }
        return;
    }
    // the row's reference, then every strip at that reference
    cmax = warp_max(cmax);
    if (lane == 0) sm_wmax[warp] = cmax;
    __syncthreads();
    cmax = sm_wmax[0];
#pragma unroll
    for (int i = 1; i < kWarps; ++i) cmax = fmaxf(cmax, sm_wmax[i]);
    double mine = 0.0;
    for (int i = i0; i < i1; ++i) { const double t = sm_S[i] * pow2_neg_d(sm_c[i] - cmax); sm_S[i] = t; mine += t; }
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) sm_warp_tot[warp] = incl;
    __syncthreads();
    double base = 0.0, R = 0.0;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) { if (i < warp) base += sm_warp_tot[i]; R += sm_warp_tot[i]; }
    int status = 0;
    if (!isfinite(R)) status = TLI_ROW_NONFINITE;            // a NaN or +inf inside the intersection
    else if (!(R > 0.0)) status = TLI_ROW_FALLBACK;          // empty intersection, or no mass in it
    if (status) {
        if (tid == 0) {
            P.draft_ids[row] = -1;
            if (P.q_out) P.q_out[row] = 0.f;
            if (P.status) P.status[row] = status;
        }
        return;
    }
    const double target = static_cast<double>(__ldg(P.u + row)) * R;
    {
        double run = base + incl - mine;                     // mass before this thread's first strip
        int cand = INT_MAX, lastpos = -1;
        for (int i = i0; i < i1; ++i) {
            const double nx = run + sm_S[i];
            if (sm_S[i] > 0.0) lastpos = i;
            if (cand == INT_MAX && nx > target) cand = i;
            run = nx;
        }
        if (cand != INT_MAX) atomicMin(&sm_found, cand);
        if (lastpos >= 0) atomicMax(&sm_lastpos, lastpos);
    }
    __syncthreads();
    const int found = sm_found;
    const int T = (found != INT_MAX) ? found : sm_lastpos;   // sm_lastpos >= 0 because R > 0
    if (T >= i0 && T < i1) {
        double before = base + incl - mine;
        for (int i = i0; i < T; ++i) before += sm_S[i];
        // what is left of the target inside strip T, in the strip's own scale; when rounding left
        // no strip above the target the walk below ends on the last positive element
        sm_rem = (found != INT_MAX) ? scale_up(target - before, cmax - sm_c[T]) : INFINITY;
        sm_total = R;
    }
    __syncthreads();
    if (warp != 0) return;

    // ---- warp 0 walks strip T ----
    const double rem = sm_rem;
    const float s = 1.4426950408889634f / tau;
    const float cT = sm_c[T];
    const int nvec = rv.nvec();
    uint4 m[kVecPerThread];
    float vs[kVecPerThread];
    {
        uint32_t bits[kVecPerThread];
        draft_load_strip<DT>(P, rv, T, nvec, lane, m, bits);
    }
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        float w[EPV];
        vs[k] = draft_vector_sum<DT>(m[k], s, -cT, w);
    }
    // vector g = k*32 + lane in address order: mass before it, fp64
    double carry = 0.0;
    int cand = INT_MAX, lastpos = -1;
    double pre_of_cand = 0.0;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const double mine_v = static_cast<double>(vs[k]);
        double inc = mine_v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += up;
        }
        const double pre = carry + inc - mine_v;
        if (vs[k] > 0.f) lastpos = k * 32 + lane;
        if (cand == INT_MAX && pre + mine_v > rem) { cand = k * 32 + lane; pre_of_cand = pre; }
        carry += __shfl_sync(0xffffffffu, inc, 31);
    }
    const int gfound = __reduce_min_sync(0xffffffffu, cand);
    const int glast = __reduce_max_sync(0xffffffffu, lastpos);
    const int G = (gfound != INT_MAX) ? gfound : glast;
    if (G < 0) {                                             // cannot happen when the strip has positive mass
        if (lane == 0) {
            P.draft_ids[row] = -1;
            if (P.q_out) P.q_out[row] = 0.f;
            if (P.status) P.status[row] = TLI_ROW_FALLBACK;
        }
        return;
    }
    if (lane == (G & 31)) {
        const double rem2 = (gfound != INT_MAX) ? (rem - pre_of_cand) : INFINITY;
        float w[EPV];
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k)
            if (k == (G >> 5)) draft_vector_sum<DT>(m[k], s, -cT, w);
        float runf = 0.f, wp = w[0];
        int pick = -1, lastw = 0;
#pragma unroll
        for (int i = 0; i < EPV; ++i) {
            runf = (i == 0) ? w[0] : __fadd_rn(runf, w[i]);
            if (w[i] > 0.f) lastw = i;
            if (pick < 0 && static_cast<double>(runf) > rem2) pick = i;
        }
        if (pick < 0) pick = lastw;
#pragma unroll
        for (int i = 1; i < EPV; ++i) wp = (i == pick) ? w[i] : wp;
        int id = rv.first_elem(T * (32 * kVecPerThread) + G) + pick;
        id = min(max(id, 0), P.V_d - 1);
        P.draft_ids[row] = id;
        if (P.q_out) P.q_out[row] = static_cast<float>(static_cast<double>(wp) * pow2_neg_d(cT - cmax) / sm_total);
        if (P.status) P.status[row] = 0;
    }
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 6) tli_draft_kernel(const DraftParams P) {
    constexpr int EPV = Elt<DT>::kPerVec;
    __shared__ int sm_last;
    const int row = blockIdx.y, tile = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = row / P.R, r = row - b * P.R;
    const float tau = __ldg(P.tau + b);
    if (!(tau >= 0.f) || isinf(tau)) {
        if (tile == 0 && tid == 0) {
            P.draft_ids[row] = -1;
            if (P.q_out) P.q_out[row] = 0.f;
            if (P.status) P.status[row] = TLI_ROW_BAD_TEMPERATURE;
        }
        return;
    }
    if (P.lengths && r > max(__ldg(P.lengths + b), 0)) {        // not a row of this sequence
        if (tile == 0 && tid == 0) {
            P.draft_ids[row] = -1;
            if (P.q_out) P.q_out[row] = 0.f;
            if (P.status) P.status[row] = 0;
        }
        return;
    }
    const RowView<DT> rv(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(r) * P.d_sr, P.V_d);
    const int nvec = rv.nvec();
    const int strip = tile * kStripsPerTile + warp;

    uint4 m[kVecPerThread];
    uint32_t bits[kVecPerThread];
    draft_load_strip<DT>(P, rv, strip, nvec, lane, m, bits);
    DraftPart pt;
    if (tau == 0.f) {
        // largest logit inside the intersection, lowest id; an id inside it counts even at -inf
        float best = -INFINITY; int idx = INT_MAX; bool bad = false;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            float z[EPV];
            unpack<DT>(m[k], z);
            const int e0 = rv.first_elem(strip * (32 * kVecPerThread) + k * 32 + lane);
#pragma unroll
            for (int i = 0; i < EPV; ++i)
                if ((bits[k] >> i) & 1u) {
                    bad = bad || !(z[i] < INFINITY);
                    if (idx == INT_MAX || z[i] > best) { best = z[i]; idx = e0 + i; }
                }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float b2 = __shfl_xor_sync(0xffffffffu, best, o);
            const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
            if (better(b2, i2, best, idx)) { best = b2; idx = i2; }
        }
        pt.S = static_cast<double>(idx); pt.c = best;
        pt.flags = __any_sync(0xffffffffu, bad) ? static_cast<int>(TLI_ROW_NONFINITE) : 0;
    } else {
        const float s = 1.4426950408889634f / tau;
        float mx;
        if constexpr (DT == TLI_BF16) {
            uint32_t mm = bf16x2_max(bf16x2_max(m[0].x, m[0].y), bf16x2_max(m[0].z, m[0].w));
#pragma unroll
            for (int k = 1; k < kVecPerThread; ++k)
                mm = bf16x2_max(mm, bf16x2_max(bf16x2_max(m[k].x, m[k].y), bf16x2_max(m[k].z, m[k].w)));
            mx = fmaxf(bf16_lo(mm), bf16_hi(mm));
        } else {
            mx = -INFINITY;
#pragma unroll
            for (int k = 0; k < kVecPerThread; ++k)
                mx = fmaxf(mx, fmaxf(fmaxf(__uint_as_float(m[k].x), __uint_as_float(m[k].y)),
                                     fmaxf(__uint_as_float(m[k].z), __uint_as_float(m[k].w))));
        }
        const float c = reference_for(warp_max(mx) * s);
        double acc = 0.0;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            float w[EPV];
            acc += static_cast<double>(draft_vector_sum<DT>(m[k], s, -c, w));
        }
        pt.S = warp_sum(acc); pt.c = c; pt.flags = 0;
    }
    if (lane == 0 && strip < P.nstrip) {
        store_part(P.part + static_cast<size_t>(row) * P.nstrip + strip, pt);
        if (!P.split) __threadfence();
    }
    if (P.split) return;
    __syncthreads();
    if (tid == 0) {
        const unsigned ticket = atomicAdd(P.cnt + row, 1u);
        sm_last = (ticket == static_cast<unsigned>(P.ntile) - 1);
        if (sm_last) P.cnt[row] = 0;
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    draft_select<DT>(P, row, rv, tau);
}

// Large batches: the selections as a kernel of their own, one CTA per row, so that the tile CTAs
// carry neither a fence nor a ticket.
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_draft_select_kernel(const DraftParams P) {
    const int row = blockIdx.x;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = row / P.R, r = row - b * P.R;
    const float tau = __ldg(P.tau + b);
    if (!(tau >= 0.f) || isinf(tau)) return;                 // the tile kernel has written this row
    if (P.lengths && r > max(__ldg(P.lengths + b), 0)) return;   // this one too
    const RowView<DT> rv(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(r) * P.d_sr, P.V_d);
    draft_select<DT>(P, row, rv, tau);
}

// Algorithm 2's comparison: the drafts re-tokenised into target ids against the tokens sampled from
// the target rows; one thread per sequence.
struct SlemParams {
    int B, M;
    const int *candidates; const int *lengths; const float *tau;
    int *sampled;              // [B, M+1], written by the sampling kernels
    const int *row_flags;      // [B, M+1]
    int *accepted; int *next_token; int *status;
};
__global__ void __launch_bounds__(128) tli_slem_match_kernel(const SlemParams P) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= P.B) return;
    const float tau = __ldg(P.tau + b);
    int m = P.lengths ? __ldg(P.lengths + b) : P.M;
    m = min(max(m, 0), P.M);
    int *t = P.sampled + static_cast<size_t>(b) * (P.M + 1);
    int flags = 0;
    if (!(tau >= 0.f) || isinf(tau)) flags = TLI_ROW_BAD_TEMPERATURE;
    else for (int j = 0; j <= m; ++j) flags |= __ldcg(P.row_flags + static_cast<size_t>(b) * (P.M + 1) + j);
    int n = 0, next = 0;
    if (flags) {
        for (int j = 0; j <= P.M; ++j) t[j] = -1;
    } else {
        n = m;
        for (int j = 0; j < m; ++j)
            if (__ldcg(t + j) != __ldg(P.candidates + static_cast<size_t>(b) * P.M + j)) { n = j; break; }
        next = __ldcg(t + n);
    }
    P.accepted[b] = n;
    P.next_token[b] = next;
    if (P.status) P.status[b] = flags;
}

// ---------------------------------------------------------------------------
// expected acceptance rates of every draft position (the paper's table of expected acceptance rates)
// ---------------------------------------------------------------------------
//
// Three small steps.  (1) Strip statistics of the K target rows and the K drafter rows of every
// sequence: reference and sum of 2^(z*s - c), for drafter rows once over all of D and once over the
// intersection (same reference).  (2) One CTA per row folds its strips.  (3) One CTA per 16 KB tile
// of a drafter row walks the ids inside the intersection, gathers the target logit at map[x] and
// adds min{p, q} and min{p, q'}; the last CTA of the pair (atomic ticket) adds the tiles in order.

struct __align__(16) RateStrip {       // per strip of a row
    double s_all, s_in;                // sums at reference c (temperature 0: best ids, all / inside)
    float c, c_in;                     // reference (temperature 0: largest logit, all / inside)
    int flags, pad;
};
struct __align__(16) RateRow {         // per row
    double s_all, s_in;
    float c, pad0;
    int idx_all, idx_in, flags, pad1;
};
struct RateParams {
    int B, K, V_t, V_d;
    const void *zt; long long t_sb, t_sk;
    const void *zd; long long d_sb, d_sk;
    const int *map; const uint32_t *maskbits; const float *tau;
    float *mass, *alpha_union, *alpha_tli; int *status;
    RateStrip *strips;     // [2*B*K][nstrip_max]
    RateRow *rows;         // [2*B*K]: target rows first, then drafter rows
    double2 *tiles;        // [B*K][ntile_d]
    unsigned *cnt;         // [B*K] tickets, zero between calls
    int nstrip_t, nstrip_d, nstrip_max, ntile_d;
};

// grid (tiles of the longer kind of row, 2*B*K): blockIdx.y < B*K target rows, then drafter rows
template <int DT>
__global__ void __launch_bounds__(kThreads, 6) tli_rate_stats_kernel(const RateParams P) {
    constexpr int EPV = Elt<DT>::kPerVec;
    const int BK = P.B * P.K;
    const int row = blockIdx.y;
    const bool drafter = row >= BK;
    const int pair = drafter ? row - BK : row;
    const int b = pair / P.K, j = pair - b * P.K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int strip = blockIdx.x * kStripsPerTile + warp;
    if (strip >= (drafter ? P.nstrip_d : P.nstrip_t)) return;
    const float tau = __ldg(P.tau + b);
    if (!(tau >= 0.f) || isinf(tau)) return;
    const RowView<DT> rv = drafter
        ? RowView<DT>(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(j) * P.d_sk, P.V_d)
        : RowView<DT>(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(j) * P.t_sk, P.V_t);
    const int nvec = rv.nvec();
    float z[kVecPerThread][EPV];
    uint32_t in_row[kVecPerThread], in_map[kVecPerThread];
    const int v0 = strip * (32 * kVecPerThread);
    const bool interior = rv.first_elem(v0) >= 0 && rv.first_elem(v0 + 32 * kVecPerThread - 1) + EPV <= rv.V;
    if (interior) {                                   // the whole strip inside the row: no per-vector tests
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int v = v0 + k * 32 + lane;
            unpack<DT>(__ldg(rv.vec0 + v), z[k]);
            in_row[k] = (1u << EPV) - 1u;
            in_map[k] = drafter ? (mask_bits(P.maskbits, rv.first_elem(v)) & in_row[k]) : 0u;
        }
    } else
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int v = strip * (32 * kVecPerThread) + k * 32 + lane;
        in_row[k] = 0u; in_map[k] = 0u;
        if (v < nvec) {
            const int e0 = rv.first_elem(v);
            unpack<DT>(rv.load(v), z[k]);
            in_row[k] = (1u << EPV) - 1u;
            if (e0 < 0) in_row[k] &= ~((1u << (-e0)) - 1u);
            if (e0 + EPV > rv.V) in_row[k] &= (1u << (rv.V - e0)) - 1u;
            if (drafter) in_map[k] = mask_bits(P.maskbits, e0) & in_row[k];
        } else {
#pragma unroll
            for (int i = 0; i < EPV; ++i) z[k][i] = -INFINITY;
        }
    }
    RateStrip out;
    out.pad = 0;
    if (tau == 0.f) {
        float ba = -INFINITY, bi = -INFINITY; int ia = INT_MAX, ii = INT_MAX; bool bad = false;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const int e0 = rv.first_elem(strip * (32 * kVecPerThread) + k * 32 + lane);
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                if ((in_row[k] >> i) & 1u) {
                    bad = bad || !(z[k][i] < INFINITY);
                    if (ia == INT_MAX || z[k][i] > ba) { ba = z[k][i]; ia = e0 + i; }
                }
                if ((in_map[k] >> i) & 1u) { if (ii == INT_MAX || z[k][i] > bi) { bi = z[k][i]; ii = e0 + i; } }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float b2 = __shfl_xor_sync(0xffffffffu, ba, o); int i2 = __shfl_xor_sync(0xffffffffu, ia, o);
            if (better(b2, i2, ba, ia)) { ba = b2; ia = i2; }
            b2 = __shfl_xor_sync(0xffffffffu, bi, o); i2 = __shfl_xor_sync(0xffffffffu, ii, o);
            if (better(b2, i2, bi, ii)) { bi = b2; ii = i2; }
        }
        out.s_all = static_cast<double>(ia); out.s_in = static_cast<double>(ii); out.c = ba; out.c_in = bi;
        out.flags = __any_sync(0xffffffffu, bad) ? static_cast<int>(TLI_ROW_NONFINITE) : 0;
    } else {
        const float s = 1.4426950408889634f / tau;
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k)
#pragma unroll
            for (int i = 0; i < EPV; ++i) mx = fmaxf(mx, z[k][i]);
        const float c = reference_for(warp_max(mx) * s);
        double sa = 0.0, si = 0.0;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            float wa = 0.f, wi = 0.f;
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                const float w = ex2(__fmaf_rn(z[k][i], s, -c));        // -inf outside the row: 0
                wa = __fadd_rn(wa, w);
                wi = __fadd_rn(wi, ((in_map[k] >> i) & 1u) ? w : 0.f);
            }
            sa += static_cast<double>(wa); si += static_cast<double>(wi);
        }
        out.s_all = warp_sum(sa); out.s_in = warp_sum(si); out.c = c; out.c_in = c; out.flags = 0;
    }
    if (lane == 0) {
        const double2 *src = reinterpret_cast<const double2 *>(&out);
        double2 *dst = reinterpret_cast<double2 *>(P.strips + static_cast<size_t>(row) * P.nstrip_max + strip);
        __stcg(dst, src[0]); __stcg(dst + 1, src[1]);
    }
}

// one CTA of 128 threads per row: the strips of a row at one reference, in strip order per thread
__global__ void __launch_bounds__(128) tli_rate_rows_kernel(const RateParams P) {
    __shared__ float sm_c[4]; __shared__ int sm_i[4], sm_i2[4]; __shared__ float sm_c2[4];
    __shared__ double sm_a[4], sm_b[4]; __shared__ int sm_flags;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int BK = P.B * P.K;
    const int row = blockIdx.x;
    const bool drafter = row >= BK;
    const int pair = drafter ? row - BK : row;
    const int b = pair / P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float tau = __ldg(P.tau + b);
    if (!(tau >= 0.f) || isinf(tau)) return;
    const int nstrip = drafter ? P.nstrip_d : P.nstrip_t;
    const RateStrip *src = P.strips + static_cast<size_t>(row) * P.nstrip_max;
    if (tid == 0) sm_flags = 0;
    __syncthreads();
    RateRow out;
    out.pad0 = 0.f; out.pad1 = 0; out.idx_all = INT_MAX; out.idx_in = INT_MAX; out.s_all = 0.0; out.s_in = 0.0; out.c = kNegBig;
    int flags = 0;
    if (tau == 0.f) {
        float ba = -INFINITY, bi = -INFINITY; int ia = INT_MAX, ii = INT_MAX;
        for (int i = tid; i < nstrip; i += 128) {
            const double2 lo = __ldcg(reinterpret_cast<const double2 *>(src + i));
            const double2 hi = __ldcg(reinterpret_cast<const double2 *>(src + i) + 1);
            const float2 cc = *reinterpret_cast<const float2 *>(&hi.x);
            flags |= reinterpret_cast<const int2 *>(&hi.y)->x;
            const int a2 = static_cast<int>(lo.x), i2 = static_cast<int>(lo.y);
            if (better(cc.x, a2, ba, ia)) { ba = cc.x; ia = a2; }
            if (better(cc.y, i2, bi, ii)) { bi = cc.y; ii = i2; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float b2 = __shfl_xor_sync(0xffffffffu, ba, o); int i2 = __shfl_xor_sync(0xffffffffu, ia, o);
            if (better(b2, i2, ba, ia)) { ba = b2; ia = i2; }
            b2 = __shfl_xor_sync(0xffffffffu, bi, o); i2 = __shfl_xor_sync(0xffffffffu, ii, o);
            if (better(b2, i2, bi, ii)) { bi = b2; ii = i2; }
        }
        if (lane == 0) { sm_c[warp] = ba; sm_i[warp] = ia; sm_c2[warp] = bi; sm_i2[warp] = ii; }
        if (flags) atomicOr(&sm_flags, flags);
        __syncthreads();
        if (tid == 0) {
            ba = sm_c[0]; ia = sm_i[0]; bi = sm_c2[0]; ii = sm_i2[0];
            for (int w = 1; w < 4; ++w) {
                if (better(sm_c[w], sm_i[w], ba, ia)) { ba = sm_c[w]; ia = sm_i[w]; }
                if (better(sm_c2[w], sm_i2[w], bi, ii)) { bi = sm_c2[w]; ii = sm_i2[w]; }
            }
            out.idx_all = ia; out.idx_in = ii; out.flags = sm_flags;
        }
    } else {
        float c = kNegBig;
        for (int i = tid; i < nstrip; i += 128) {
            const double2 hi = __ldcg(reinterpret_cast<const double2 *>(src + i) + 1);
            c = fmaxf(c, reinterpret_cast<const float2 *>(&hi.x)->x);
        }
        c = warp_max(c);
        if (lane == 0) sm_c[warp] = c;
        __syncthreads();
        c = fmaxf(fmaxf(sm_c[0], sm_c[1]), fmaxf(sm_c[2], sm_c[3]));
        double sa = 0.0, si = 0.0;
        for (int i = tid; i < nstrip; i += 128) {
            const double2 lo = __ldcg(reinterpret_cast<const double2 *>(src + i));
            const double2 hi = __ldcg(reinterpret_cast<const double2 *>(src + i) + 1);
            const double f = pow2_neg_d(reinterpret_cast<const float2 *>(&hi.x)->x - c);
            sa += lo.x * f; si += lo.y * f;
        }
        sa = warp_sum(sa); si = warp_sum(si);
        if (lane == 0) { sm_a[warp] = sa; sm_b[warp] = si; }
        __syncthreads();
        if (tid == 0) {
            out.s_all = ((sm_a[0] + sm_a[1]) + sm_a[2]) + sm_a[3];
            out.s_in = ((sm_b[0] + sm_b[1]) + sm_b[2]) + sm_b[3];
            out.c = c;
            out.flags = (!isfinite(out.s_all) || !(out.s_all > 0.0)) ? static_cast<int>(TLI_ROW_NONFINITE) : 0;
        }
    }
    if (tid == 0) {
        const double2 *w = reinterpret_cast<const double2 *>(&out);
        double2 *dst = reinterpret_cast<double2 *>(P.rows + row);
        __stcg(dst, w[0]); __stcg(dst + 1, w[1]); __stcg(dst + 2, w[2]);
    }
}

__device__ __forceinline__ RateRow load_rate_row(const RateRow *p) {
    RateRow r;
    double2 *w = reinterpret_cast<double2 *>(&r);
    w[0] = __ldcg(reinterpret_cast<const double2 *>(p));
    w[1] = __ldcg(reinterpret_cast<const double2 *>(p) + 1);
    w[2] = __ldcg(reinterpret_cast<const double2 *>(p) + 2);
    return r;
}

// grid (ntile_d, B*K)
template <int DT>
__global__ void __launch_bounds__(kThreads, 6) tli_rate_pairs_kernel(const RateParams P) {
    constexpr int EPV = Elt<DT>::kPerVec;
    __shared__ double sm_u[kWarps], sm_t[kWarps];
    __shared__ int sm_last;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int pair = blockIdx.y, tile = blockIdx.x;
    const int b = pair / P.K, j = pair - b * P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float tau = __ldg(P.tau + b);
    const int BK = P.B * P.K;
    if (!(tau >= 0.f) || isinf(tau)) {
        if (tile == 0 && tid == 0) {
            P.mass[pair] = 0.f; P.alpha_union[pair] = 0.f; P.alpha_tli[pair] = 0.f;
            if (P.status) P.status[pair] = TLI_ROW_BAD_TEMPERATURE;
        }
        return;
    }
    const RateRow rt = load_rate_row(P.rows + pair);
    const RateRow rd = load_rate_row(P.rows + BK + pair);
    int status = rt.flags | rd.flags;
    if (tau == 0.f) {
        if (tile == 0 && tid == 0) {
            float M = 0.f, au = 0.f, at = 0.f;
            if (!(status & TLI_ROW_NONFINITE)) {
                const int t_all = (rd.idx_all != INT_MAX) ? __ldg(P.map + rd.idx_all) : -1;
                const int t_in = (rd.idx_in != INT_MAX) ? __ldg(P.map + rd.idx_in) : -1;
                M = t_all >= 0 ? 1.f : 0.f;
                au = (t_all >= 0 && t_all == rt.idx_all) ? 1.f : 0.f;
                at = (t_in >= 0 && t_in == rt.idx_all) ? 1.f : 0.f;
                if (rd.idx_in == INT_MAX) status |= TLI_ROW_FALLBACK;
            }
            P.mass[pair] = M; P.alpha_union[pair] = au; P.alpha_tli[pair] = at;
            if (P.status) P.status[pair] = status;
        }
        return;
    }
    if (status & TLI_ROW_NONFINITE) {
        if (tile == 0 && tid == 0) {
            P.mass[pair] = 0.f; P.alpha_union[pair] = 0.f; P.alpha_tli[pair] = 0.f;
            if (P.status) P.status[pair] = TLI_ROW_NONFINITE;
        }
        return;
    }
    const float s = 1.4426950408889634f / tau;
    const float rs_t = static_cast<float>(1.0 / rt.s_all);
    const float rs_a = static_cast<float>(1.0 / rd.s_all);
    const float rs_i = rd.s_in > 0.0 ? static_cast<float>(1.0 / rd.s_in) : 0.f;     // q' = e / S_in
    const RowView<DT> rv(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(j) * P.d_sk, P.V_d);
    const long long t_off = static_cast<long long>(b) * P.t_sb + static_cast<long long>(j) * P.t_sk;
    const int nvec = rv.nvec();
    double au = 0.0, at = 0.0;
    const int v_first = tile * kVecPerTile;
    const bool lean = (rv.head & 3) == 0 && rv.first_elem(v_first) >= 0 &&
                      rv.first_elem(v_first + kVecPerTile - 1) + EPV <= rv.V;     // the same for the whole CTA
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int v = v_first + k * kThreads + tid;
        if (!lean && v >= nvec) continue;
        const int e0 = rv.first_elem(v);
        float z[EPV];
        int tmap[EPV];
        if (lean) {                                   // whole tile inside an aligned row: vector loads, no range tests
            unpack<DT>(__ldg(rv.vec0 + v), z);
#pragma unroll
            for (int i = 0; i < EPV; i += 4) {
                const int4 q = __ldg(reinterpret_cast<const int4 *>(P.map + e0 + i));
                tmap[i] = q.x; tmap[i + 1] = q.y; tmap[i + 2] = q.z; tmap[i + 3] = q.w;
            }
        } else {
            unpack<DT>(rv.load(v), z);
#pragma unroll
            for (int i = 0; i < EPV; ++i) tmap[i] = (e0 + i >= 0 && e0 + i < P.V_d) ? __ldg(P.map + e0 + i) : -1;
        }
        float su = 0.f, st = 0.f;
#pragma unroll
        for (int i = 0; i < EPV; ++i) {
            if (tmap[i] >= 0) {
                const int t = tmap[i];
                const float ed = ex2(__fmaf_rn(z[i], s, -rd.c));
                const float et = ex2(__fmaf_rn(load_elt<DT>(P.zt, t_off + t), s, -rt.c));
                const float p = __fmul_rn(et, rs_t);
                su = __fadd_rn(su, fminf(p, __fmul_rn(ed, rs_a)));
                st = __fadd_rn(st, fminf(p, __fmul_rn(ed, rs_i)));
            }
        }
        au += static_cast<double>(su); at += static_cast<double>(st);
    }
    au = warp_sum(au); at = warp_sum(at);
    if (lane == 0) { sm_u[warp] = au; sm_t[warp] = at; }
    __syncthreads();
    if (tid == 0) {
        double u2 = 0.0, t2 = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { u2 += sm_u[w]; t2 += sm_t[w]; }
        __stcg(P.tiles + static_cast<size_t>(pair) * P.ntile_d + tile, make_double2(u2, t2));
        __threadfence();
        const unsigned ticket = atomicAdd(P.cnt + pair, 1u);
        sm_last = (ticket == static_cast<unsigned>(P.ntile_d) - 1);
        if (sm_last) P.cnt[pair] = 0;
    }
    __syncthreads();
    if (!sm_last || tid != 0) return;
    __threadfence();
    double u2 = 0.0, t2 = 0.0;
    for (int i = 0; i < P.ntile_d; ++i) {
        const double2 v = __ldcg(P.tiles + static_cast<size_t>(pair) * P.ntile_d + i);
        u2 += v.x; t2 += v.y;
    }
    const double M = rd.s_in / rd.s_all;
    if (!(rd.s_in > 0.0)) status |= TLI_ROW_FALLBACK;          // empty intersection, or no mass in it
    P.mass[pair] = static_cast<float>(M);
    P.alpha_union[pair] = static_cast<float>(u2);
    P.alpha_tli[pair] = static_cast<float>(t2);
    if (P.status) P.status[pair] = status;
}

// ---------------------------------------------------------------------------
// vocabulary-sharded verification (the logits of a tensor-parallel LM head)
// ---------------------------------------------------------------------------
//
// Every shard holds a slice of each target row and of each drafter row.  Algorithm 4's
// denominator (the sum over the intersection) and Algorithm 5's residual normaliser are the two
// sums that cross shards; everything else is local:
//   statistics   the statistics kernel on the slices, then one record per sequence: (reference,
//                sum) of each of its 2K+1 rows over this shard's ids, and the logits of the drafted
//                tokens that this shard owns.                         -> exchanged (all-gather)
//   decision     every shard folds the records of all shards (exact powers of two, fp64) and takes
//                Algorithm 5's decisions: the same on every shard.  It then packs its slice of
//                drafter row n of every sequence that rejected a draft.  -> exchanged (all-gather)
//   weights      tile sums of max(0, p - q'_T) and of p over this shard's target ids, q' read from
//                the gathered drafter row, and their totals.              -> exchanged (all-gather)
//   selection    every shard adds the totals in shard order; the shard that holds v * total walks
//                its tiles, the others report -1.                    -> combined (maximum)
// The exchanges are the caller's (NCCL through torch.distributed); these kernels read and write
// local memory only.

// doubles per sequence of one shard's record: (reference | max, sum | arg-max) per row, then the
// target and the drafter logit of every drafted token (0 where another shard owns it)
__host__ __device__ inline int shard_record_len(int K) { return 2 * (2 * K + 1) + 2 * K; }

struct ShardParams {
    Params P;
    int G, g;            // shards, this shard
    int wt, wd;          // target / drafter ids per shard (the last shards may hold fewer, or none)
    int V_t_all, V_d_all;
    double *record;            // this shard's record [B][shard_record_len(K)]
    const double *records;     // all shards' records [G][B][shard_record_len(K)]
    void *rows_out;            // this shard's slices of drafter row n [B][row_pitch elements]
    const void *rows_all;      // all shards' [G][B][row_pitch]
    int row_pitch;
    double *mass;              // this shard's totals [B][2]: residual, p
    const double *masses;      // all shards' [G][B][2]
};

// One CTA per sequence: the shard's segment partials folded per row into its record, and the
// logits of the drafted tokens that live on this shard.
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_shard_fold_kernel(const ShardParams S) {
    const Params &P = S.P;
    const int b = blockIdx.x, tid = threadIdx.x, K = P.K;
    const float tau = __ldg(P.tau + b);
    double *rec = S.record + static_cast<size_t>(b) * shard_record_len(K);
    const bool bad = !(tau >= 0.f) || isinf(tau);
    const bool greedy = (tau == 0.f);
    if (tid < K) {                                   // the drafted tokens this shard owns
        double zt = 0.0, zd = 0.0;
        const int x = __ldg(P.draft + static_cast<size_t>(b) * K + tid);
        if (!bad && !greedy && x >= 0 && x < S.V_d_all) {
            const int t = __ldg(P.map + x);
            if (t >= P.t_begin && t < P.t_begin + P.V_t)
                zt = load_elt<DT>(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(tid) * P.t_sk + (t - P.t_begin));
            if (t >= 0 && x >= P.d_begin && x < P.d_begin + P.V_d)
                zd = load_elt<DT>(P.zd, static_cast<long long>(b) * P.d_sb + static_cast<long long>(tid) * P.d_sk + (x - P.d_begin));
        }
        rec[2 * (2 * K + 1) + tid] = zt;
        rec[2 * (2 * K + 1) + K + tid] = zd;
    }
    const int nrows = 2 * K + 1;
    for (int r0 = 0; r0 < nrows; r0 += kThreads / 8) {
        const int r = r0 + (tid >> 3);
        const int sub = tid & 7;
        const bool is_t = r <= K;
        const bool mine = r < nrows && !bad && !(greedy && !is_t);
        const int nseg = !mine ? 0 : (is_t ? P.nst : P.nsd);
        const float2 *part = is_t ? P.part_t + (static_cast<size_t>(b) * (K + 1) + r) * P.nst
                                  : P.part_d + (static_cast<size_t>(b) * K + (r - K - 1)) * P.nsd;
        if (greedy) {
            float best = -INFINITY; int idx = INT_MAX;
            for (int i = sub; i < nseg; i += 8) {
                float2 pr = __ldcg(part + i);
                int i2 = __float_as_int(pr.y);
                if (pr.x > best || (pr.x == best && i2 < idx)) { best = pr.x; idx = i2; }
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                float b2 = __shfl_xor_sync(0xffffffffu, best, o);
                int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                if (b2 > best || (b2 == best && i2 < idx)) { best = b2; idx = i2; }
            }
            if (sub == 0 && r < nrows) { rec[2 * r] = static_cast<double>(best); rec[2 * r + 1] = static_cast<double>(idx); }
        } else {
            float c = kNegBig;
            double sum = 0.0;
            for (int i = sub; i < nseg; i += 8) {
                const float2 pr = __ldcg(part + i);
                const float cn = fmaxf(c, pr.x);
                sum = sum * pow2_neg_d(c - cn) + static_cast<double>(pr.y) * pow2_neg_d(pr.x - cn);
                c = cn;
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                const float c2 = __shfl_xor_sync(0xffffffffu, c, o);
                const double s2 = __shfl_xor_sync(0xffffffffu, sum, o);
                const float cn = fmaxf(c, c2);
                sum = sum * pow2_neg_d(c - cn) + s2 * pow2_neg_d(c2 - cn);
                c = cn;
            }
            if (sub == 0 && r < nrows) { rec[2 * r] = static_cast<double>(c); rec[2 * r + 1] = sum; }
        }
    }
}

// One CTA per sequence, the same on every shard: the records of all shards folded in shard order,
// Algorithm 5's acceptance tests and count, the hand-over to the weights pass.
__global__ void __launch_bounds__(128) tli_shard_decide_kernel(const ShardParams S) {
    const Params &P = S.P;
    const int b = blockIdx.x, tid = threadIdx.x, K = P.K, G = S.G;
    const int len = shard_record_len(K);
    __shared__ double sm_c[2 * TLI_MAX_K + 1], sm_s[2 * TLI_MAX_K + 1];
    __shared__ int sm_accept[TLI_MAX_K];
    __shared__ int sm_flags;
    const float tau = __ldg(P.tau + b);
    if (tid == 0) sm_flags = 0;
    if (!(tau >= 0.f) || isinf(tau)) {
        if (tid == 0) {
            P.accepted[b] = 0; P.next_token[b] = 0;
            if (P.status) P.status[b] = TLI_ROW_BAD_TEMPERATURE;
            RowSel rs = {0, MODE_SKIP, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            P.sel[b] = rs;
        }
        if (tid < K) {
            if (P.p_out) P.p_out[static_cast<size_t>(b) * K + tid] = 0.f;
            if (P.q_out) P.q_out[static_cast<size_t>(b) * K + tid] = 0.f;
        }
        return;
    }
    const bool greedy = (tau == 0.f);
    const int nrows = greedy ? K + 1 : 2 * K + 1;
    for (int r = tid; r < nrows; r += blockDim.x) {
        if (greedy) {
            double best = -INFINITY, idx = static_cast<double>(INT_MAX);
            for (int g = 0; g < G; ++g) {
                const double *rec = S.records + (static_cast<size_t>(g) * P.B + b) * len;
                const double m = rec[2 * r], i2 = rec[2 * r + 1];
                if (m > best || (m == best && i2 < idx)) { best = m; idx = i2; }
            }
            sm_c[r] = best; sm_s[r] = (idx == static_cast<double>(INT_MAX)) ? 0.0 : idx;
        } else {
            double c = static_cast<double>(kNegBig), sum = 0.0;
            for (int g = 0; g < G; ++g) {
                const double *rec = S.records + (static_cast<size_t>(g) * P.B + b) * len;
                const double c2 = rec[2 * r], s2 = rec[2 * r + 1];
                const double cn = fmax(c, c2);
                sum = sum * pow2_neg_d(static_cast<float>(c - cn)) + s2 * pow2_neg_d(static_cast<float>(c2 - cn));
                c = cn;
            }
            sm_c[r] = c; sm_s[r] = sum;
        }
    }
    __syncthreads();
    const float s_f = 1.4426950408889634f / tau;
    if (tid < K) {
        const int j = tid;
        int ok = 0, fl = (P.n_mapped == 0 && !greedy) ? TLI_ROW_FALLBACK : 0;
        float pv = 0.f, qv = 0.f;
        const int x = __ldg(P.draft + static_cast<size_t>(b) * K + j);
        int t = -1;
        if (x < 0 || x >= S.V_d_all) fl |= TLI_ROW_DRAFT_RANGE;
        else { t = __ldg(P.map + x); if (t < 0) fl |= TLI_ROW_DRAFT_UNMAPPED; }
        if (greedy) {
            ok = (t >= 0 && t == static_cast<int>(sm_s[j]));
        } else {
            const double S_t = sm_s[j], S_d = sm_s[K + 1 + j];
            if (!(S_t > 0.0) || !isfinite(S_t) || !isfinite(S_d)) fl |= TLI_ROW_NONFINITE;
            else if (t >= 0) {
                const int gt = t / S.wt, gd = x / S.wd;                   // the shards that own the two logits
                const double zt = S.records[(static_cast<size_t>(gt) * P.B + b) * len + 2 * (2 * K + 1) + j];
                const double zd = S.records[(static_cast<size_t>(gd) * P.B + b) * len + 2 * (2 * K + 1) + K + j];
                const double sd = static_cast<double>(s_f);
                const double p = exp2(zt * sd - sm_c[j]) / S_t;
                const double q = (S_d > 0.0) ? exp2(zd * sd - sm_c[K + 1 + j]) / S_d : 0.0;
                double thr;
                if (q > 0.0) thr = fmin(1.0, p / q);
                else thr = (p > 0.0) ? 1.0 : 0.0;
                ok = static_cast<double>(__ldg(P.u + static_cast<size_t>(b) * (K + 1) + j)) < thr;
                pv = static_cast<float>(p); qv = static_cast<float>(q);
            }
        }
        sm_accept[j] = ok;
        if (fl) atomicOr(&sm_flags, fl);
        if (P.p_out) P.p_out[static_cast<size_t>(b) * K + j] = pv;
        if (P.q_out) P.q_out[static_cast<size_t>(b) * K + j] = qv;
    }
    __syncthreads();
    if (tid == 0) {
        int n = K;
        for (int j = 0; j < K; ++j) if (!sm_accept[j]) { n = j; break; }
        int fl = sm_flags;
        if (!greedy) {
            const double S_n = sm_s[n];
            if (!(S_n > 0.0) || !isfinite(S_n)) fl |= TLI_ROW_NONFINITE;
        }
        RowSel rs;
        rs.n = n; rs.mode = MODE_SKIP; rs.s = s_f; rs.c_t = 0.f; rs.rs_t = 0.f; rs.c_d = 0.f; rs.rs_d = 0.f;
        rs.v = __ldg(P.u + static_cast<size_t>(b) * (K + 1) + K);
        int token = -1;                            // -1: the selection supplies it
        if (greedy) {
            token = static_cast<int>(sm_s[n]);
        } else if (fl & TLI_ROW_NONFINITE) {
            n = 0; token = 0;
        } else {
            rs.c_t = static_cast<float>(sm_c[n]);
            rs.rs_t = static_cast<float>(1.0 / sm_s[n]);
            if (n < K) {
                const double S_d = sm_s[K + 1 + n];
                rs.mode = MODE_RESIDUAL;
                rs.c_d = static_cast<float>(sm_c[K + 1 + n]);
                rs.rs_d = (S_d > 0.0) ? static_cast<float>(1.0 / S_d) : 0.f;
            } else {
                rs.mode = MODE_TARGET_ONLY;
            }
        }
        rs.n = n;
        P.accepted[b] = n;
        P.next_token[b] = token;
        if (P.status) P.status[b] = fl;
        P.sel[b] = rs;
    }
}

// This shard's slice of drafter row n of every sequence that rejected a draft, as 16-byte vectors
// (ids beyond the slice read -inf).  grid (vectors / 256, B).
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_shard_pack_kernel(const ShardParams S) {
    constexpr int EPV = Elt<DT>::kPerVec;
    const Params &P = S.P;
    const int b = blockIdx.y;
    const RowSel sel = P.sel[b];
    if (sel.mode != MODE_RESIDUAL) return;
    const int v = blockIdx.x * kThreads + threadIdx.x;
    if (v * EPV >= S.row_pitch) return;
    const char *row = reinterpret_cast<const char *>(P.zd) +
        (static_cast<long long>(b) * P.d_sb + static_cast<long long>(sel.n) * P.d_sk) * Elt<DT>::kBytes;
    uint32_t w[4] = {Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord, Elt<DT>::kNegInfWord};
    if constexpr (DT == TLI_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = v * 4 + i;
            if (e < P.V_d) w[i] = __ldg(reinterpret_cast<const uint32_t *>(row) + e);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = v * 8 + i;
            if (e < P.V_d) {
                const uint32_t h = __ldg(reinterpret_cast<const unsigned short *>(row) + e);
                w[i >> 1] = (i & 1) ? ((w[i >> 1] & 0x0000ffffu) | (h << 16)) : ((w[i >> 1] & 0xffff0000u) | h);
            }
        }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<char *>(S.rows_out) +
                                           static_cast<size_t>(b) * S.row_pitch * Elt<DT>::kBytes);
    dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
}

// One CTA per 16 KB tile of this shard's slice of target row n: the sums of max(0, p - q'_T) and
// of p over the tile (fp32 per vector, fp64 across).  grid (tiles, B).
template <int DT>
__global__ void __launch_bounds__(kThreads, 4) tli_shard_weights_kernel(const ShardParams S) {
    constexpr int EPV = Elt<DT>::kPerVec;
    const Params &P = S.P;
    __shared__ double sm_red[2][kWarps];
    const int b = blockIdx.y, tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowSel sel = P.sel[b];
    if (sel.mode == MODE_SKIP) return;
    const RowView<DT> rt(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(sel.n) * P.t_sk, P.V_t);
    const void *zd_rows = reinterpret_cast<const char *>(S.rows_all) + static_cast<size_t>(b) * S.row_pitch * Elt<DT>::kBytes;
    const int nvec = rt.nvec();
    double acc_r = 0.0, acc_p = 0.0;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int v = tile * kVecPerTile + k * kThreads + tid;
        if (v < nvec) {
            float pt[EPV], q[EPV], w[EPV];
            vector_p_q<DT, false, SRC_SHARDS>(P, sel, rt.load(v), rt.first_elem(v), zd_rows, pt, q);
#pragma unroll
            for (int i = 0; i < EPV; ++i) w[i] = fmaxf(0.f, __fsub_rn(pt[i], q[i]));
            acc_r += static_cast<double>(ordered_sum(w));
            acc_p += static_cast<double>(ordered_sum(pt));
        }
    }
    acc_r = warp_sum(acc_r);
    acc_p = warp_sum(acc_p);
    if (lane == 0) { sm_red[0][warp] = acc_r; sm_red[1][warp] = acc_p; }
    __syncthreads();
    if (tid == 0) {
        double tr = 0.0, tp = 0.0;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) { tr += sm_red[0][i]; tp += sm_red[1][i]; }
        __stcg(P.tilesum + static_cast<size_t>(b) * P.ntile + tile, tr);
        __stcg(P.tilesum_p + static_cast<size_t>(b) * P.ntile + tile, tp);
    }
}

// One thread per sequence: this shard's totals, tiles added in order.
__global__ void __launch_bounds__(128) tli_shard_mass_kernel(const ShardParams S) {
    const Params &P = S.P;
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= P.B) return;
    double r = 0.0, p = 0.0;
    if (P.sel[b].mode != MODE_SKIP) {
        for (int i = 0; i < P.ntile; ++i) {
            r += __ldcg(P.tilesum + static_cast<size_t>(b) * P.ntile + i);
            p += __ldcg(P.tilesum_p + static_cast<size_t>(b) * P.ntile + i);
        }
    }
    S.mass[2 * b] = r;
    S.mass[2 * b + 1] = p;
}

// One CTA per sequence, the same arithmetic on every shard: the totals of all shards added in
// shard order, the shard that holds v * total, and on that shard tile -> vector -> element.
template <int DT>
__global__ void __launch_bounds__(kThreads) tli_shard_select_kernel(const ShardParams S) {
    const Params &P = S.P;
    __shared__ int sm_tile, sm_mode;
    __shared__ double sm_rem;
    const int b = blockIdx.x, tid = threadIdx.x;
    RowSel sel = P.sel[b];
    if (sel.mode == MODE_SKIP) return;                   // decided and finished by the decision kernel
    if (tid == 0) {
        int kind = (sel.mode == MODE_RESIDUAL) ? 0 : 1;  // which totals: residual, or p
        double R = 0.0;
        for (int g = 0; g < S.G; ++g) R += S.masses[(static_cast<size_t>(g) * P.B + b) * 2 + kind];
        int fl = 0;
        if (kind == 0 && (!(R > 0.0) || !isfinite(R))) {  // zero residual mass: sample from p of the same position
            kind = 1; fl |= TLI_ROW_FALLBACK;
            R = 0.0;
            for (int g = 0; g < S.G; ++g) R += S.masses[(static_cast<size_t>(g) * P.B + b) * 2 + 1];
        }
        sm_mode = -1;
        if (!(R > 0.0) || !isfinite(R)) {                // no usable mass even from p: give up on the row
            P.next_token[b] = 0;
            fl |= TLI_ROW_NONFINITE;
        } else {
            const double target = static_cast<double>(sel.v) * R;
            int owner = -1, lastpos = 0;
            double before = 0.0, run = 0.0;
            for (int g = 0; g < S.G; ++g) {
                const double m = S.masses[(static_cast<size_t>(g) * P.B + b) * 2 + kind];
                const double nx = run + m;
                if (m > 0.0) lastpos = g;
                if (owner < 0 && nx > target) { owner = g; before = run; }
                run = nx;
            }
            if (owner < 0) { owner = lastpos; before = R - S.masses[(static_cast<size_t>(lastpos) * P.B + b) * 2 + kind]; }
            if (owner == S.g) {
                // this shard: which of its tiles
                const double *tiles = (kind == 0 ? P.tilesum : P.tilesum_p) + static_cast<size_t>(b) * P.ntile;
                const double rem = target - before;
                double run_t = 0.0, before_t = 0.0;
                int T = -1, last_t = 0;
                for (int i = 0; i < P.ntile; ++i) {
                    const double m = __ldcg(tiles + i);
                    const double nx = run_t + m;
                    if (m > 0.0) last_t = i;
                    if (T < 0 && nx > rem) { T = i; before_t = run_t; }
                    run_t = nx;
                }
                if (T < 0) { T = last_t; before_t = run_t - __ldcg(tiles + last_t); }
                sm_tile = T;
                sm_rem = rem - before_t;
                sm_mode = (kind == 0) ? MODE_RESIDUAL : MODE_TARGET_ONLY;
            } else {
                P.next_token[b] = -1;                    // another shard reports it
            }
        }
        if (fl && P.status) P.status[b] |= fl;
    }
    __syncthreads();
    if (sm_mode < 0) return;
    sel.mode = sm_mode;
    const RowView<DT> rt(P.zt, static_cast<long long>(b) * P.t_sb + static_cast<long long>(sel.n) * P.t_sk, P.V_t);
    const void *zd_rows = reinterpret_cast<const char *>(S.rows_all) + static_cast<size_t>(b) * S.row_pitch * Elt<DT>::kBytes;
    walk_tile<DT, true, SRC_SHARDS>(P, b, sel, rt, zd_rows, sm_tile, sm_rem);
}

// Kernels that do nothing, for tli_launch_probe(): the cost of getting a call's launches through
// the stream (launch, scheduling of the CTAs, the dependent launch, the cluster barrier) without any
// of its work.
__global__ void __launch_bounds__(kSThreads + 32, kCtasPerSm) tli_probe_first_kernel(int dummy) {
    extern __shared__ __align__(128) unsigned char probe_smem[];
    if (dummy < 0) probe_smem[threadIdx.x] = 0;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__global__ void __launch_bounds__(kFinThreads, 2) tli_probe_second_kernel(int dummy) {
    extern __shared__ __align__(16) unsigned char probe_smem2[];
    if (dummy < 0) probe_smem2[threadIdx.x] = 0;
    cluster_barrier();
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever complete,
// with a caller-chosen poll limit, and reports how the wait ended.  The kernel returns normally.
__global__ void tli_bounded_wait_kernel(unsigned limit, int *result, unsigned *scratch_error) {
    __shared__ uint64_t bar;
    __shared__ int sm_error;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        sm_error = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool completed = mbar_wait_slow(&bar, 0u, &sm_error, scratch_error, limit);
        result[0] = completed ? 0 : 1;              // 1: gave up, as it must
        result[1] = sm_error;                       // 1: the CTA-wide error flag was raised
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char *what) {
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", what, cudaGetErrorString(e));
    return TLI_ERR_CUDA;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

FastDiv make_fast_div(unsigned d) {
    FastDiv f;
    f.d = d;
    f.s = 0;
    while ((1ull << f.s) < d) ++f.s;
    f.m = static_cast<unsigned>((((1ull << f.s) - d) << 32) / d + 1);
    return f;
}

int chunks_per_row(int V, int dtype, int vec_per_chunk) {
    const long long epv = dtype == TLI_F32 ? 4 : 8;
    return static_cast<int>((static_cast<long long>(V) + epv - 1 + epv * vec_per_chunk - 1) / (epv * vec_per_chunk));
}

struct Layout {
    size_t part_t, part_d, sel, tilesum, total;
    int cv;              // vectors per consumer thread per stage of the statistics kernel (1, 2 or 4)
    int ntile;
    int seg_vec, nst, nsd;      // segments of the statistics kernel, see Params
    long long nseg;             // ... in all (the kernel numbers them in 32 bits)
    unsigned grid;
    int fin_cluster;     // CTAs per sequence of the cluster kernel; 0: the tile kernels draw the extra token
    int fin_slice;       // vectors of the target row per CTA of the cluster
    int fin_dvec;        // vectors reserved for the staged drafter row
    size_t fin_smem;     // its dynamic shared memory
};

// The cluster kernel keeps the whole drafter row and four bytes per 16-byte vector of its slice of
// the target row in shared memory.  It is used when that fits twice into an SM, or once while the
// whole batch is resident at one CTA per SM; larger vocabularies and batches go to the tile
// kernels, which are built for throughput.  Small batches get the widest cluster, so that more SMs
// share the one row.
constexpr size_t kFinSmemTwoPerSm = 100 * 1024;
constexpr size_t kFinSmemOnePerSm = 200 * 1024;
void plan_finish(Layout &L, int B, int V_t, int V_d, int dtype, int num_sms, int max_cluster) {
    L.fin_cluster = 0; L.fin_slice = 0; L.fin_dvec = 0; L.fin_smem = 0;
    const int nvec = chunks_per_row(V_t, dtype, 1);                 // vectors of a row, whatever its alignment
    const int dvec = chunks_per_row(V_d, dtype, 1);
    auto need = [&](int c) { return static_cast<size_t>(dvec) * 16 + static_cast<size_t>((nvec + c - 1) / c) * 4; };
    int C = 0;
    for (int c = 1; c <= max_cluster; c *= 2)
        if (need(c) <= kFinSmemTwoPerSm) { C = c; break; }
    if (C) {
        while (C < max_cluster && static_cast<long long>(B) * C * 2 <= 2LL * num_sms) C *= 2;
        if (static_cast<long long>(B) * C > 8LL * num_sms) return;
    } else {
        for (int c = max_cluster; c >= 1; c /= 2)
            if (need(c) <= kFinSmemOnePerSm && static_cast<long long>(B) * c <= num_sms) { C = c; break; }
        if (C == 0) return;
    }
    L.fin_cluster = C;
    L.fin_slice = (nvec + C - 1) / C;
    L.fin_dvec = dvec;
    L.fin_smem = need(C);
}

// Stage size: as large as leaves every CTA of the persistent grid (two per SM) about one stage
// (measured: the per-stage bookkeeping costs more than a few idle CTAs do).
// Segment size: a batch that gives every CTA many stages is cut into segments of up to 128 KB,
// about four per CTA (long enough to amortise the per-segment reduction; longer ones interleave the
// rows of a large batch worse).  A small batch is cut into the shortest segments that still number
// no more than the CTAs.
Layout make_layout(int B, int K, int V_t, int V_d, int dtype, int num_sms, int max_cluster = 8) {
    Layout L;
    const long long elt = dtype == TLI_F32 ? 4 : 2;
    const long long bytes = elt * B * (static_cast<long long>(K + 1) * V_t + static_cast<long long>(K) * V_d);
    const long long ctas = static_cast<long long>(kCtasPerSm) * num_sms;
    L.cv = 1;
    if (bytes >= ctas * (kSThreads * 2 * 16)) L.cv = 2;
    if (bytes >= ctas * (kSThreads * 4 * 16)) L.cv = 4;
    const int cvec = kSThreads * L.cv;                               // vectors per stage
    const int nvec_t = chunks_per_row(V_t, dtype, 1), nvec_d = chunks_per_row(V_d, dtype, 1);
    L.ntile = chunks_per_row(V_t, dtype, kVecPerTile);
    auto per_row = [](int nvec, int sv) { return (nvec + sv - 1) / sv; };
    auto count = [&](int sv) {
        return static_cast<long long>(B) * (static_cast<long long>(K + 1) * per_row(nvec_t, sv) + static_cast<long long>(K) * per_row(nvec_d, sv));
    };
    const long long stages = count(cvec);
    const int sv_cap = 16 * kSThreads;                               // 128 KB
    if (stages <= ctas * 16) {
        L.seg_vec = kSThreads;
        while (L.seg_vec < sv_cap && count(L.seg_vec) > ctas) L.seg_vec += kSThreads;
    } else {
        long long cps = stages / (ctas * 4);
        const long long cap = sv_cap / cvec;
        cps = cps < 1 ? 1 : (cps > cap ? cap : cps);
        L.seg_vec = static_cast<int>(cps) * cvec;
    }
    L.nst = per_row(nvec_t, L.seg_vec);
    L.nsd = per_row(nvec_d, L.seg_vec);
    const long long nseg = count(L.seg_vec);
    L.nseg = nseg;
    const long long grid = nseg < ctas ? nseg : ctas;
    L.grid = static_cast<unsigned>(grid);
    size_t off = 0;
    L.part_t = off; off = align_up(off + sizeof(float2) * static_cast<size_t>(B) * (K + 1) * L.nst, 256);
    L.part_d = off; off = align_up(off + sizeof(float2) * static_cast<size_t>(B) * K * L.nsd, 256);
    L.sel = off;    off = align_up(off + sizeof(RowSel) * static_cast<size_t>(B), 256);
    L.tilesum = off; off = align_up(off + sizeof(double) * static_cast<size_t>(B) * L.ntile, 256);
    L.total = off;
    plan_finish(L, B, V_t, V_d, dtype, num_sms, max_cluster);
    return L;
}

}  // namespace

constexpr size_t kCtxPartsBytes = 8u << 20;
constexpr size_t kCounterWords = 3 * (TLI_MAX_B + 1) + 8;     // per-sequence tickets (two sets, one spare), sticky error, schedulers

struct tli_ctx {
    int device;
    int32_t V_t, V_d, n_mapped;
    int *d_map;
    int *d_inv;
    uint32_t *d_mask;
    int tiled;                  // option: the extra token always by the tile kernels (default 0: by size)
    int max_cluster;            // widest cluster the device takes for the cluster kernel (16 where the driver allows it, else 8)
    int device_max_cluster;     // ... what tli_create() found; max_cluster can be narrowed by tli_set_max_cluster()
    float2 *d_parts;            // kCtxPartsBytes of partial results for the cluster form: all ones (kPartEmpty) between calls
    unsigned *d_counters;       // [3 * (TLI_MAX_B + 1) + 8], zero between calls: tickets, tickets, sequence states,
                                // sticky error, schedulers
    int num_sms;
    // vocabulary-sharded contexts (tli_shard_create); one shard holding everything otherwise
    int n_shards, shard;
    int32_t wt, wd;             // ids per shard
    int32_t t_begin, t_count, d_begin, d_count;
};

namespace {

cudaError_t launch_stats(const Params &P, const Layout &L, int dtype, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1; cfg.stream = stream;
    cfg.gridDim = dim3(L.grid); cfg.blockDim = dim3(kSThreads + 32); cfg.dynamicSmemBytes = kStatsSmemBytes;
    cudaError_t e = cudaSuccess;
#define TLI_LAUNCH_STATS(DT, CV) e = cudaLaunchKernelEx(&cfg, tli_stats_kernel<DT, CV>, P)
    if (dtype == TLI_F32) {
        if (L.cv == 4) TLI_LAUNCH_STATS(TLI_F32, 4); else if (L.cv == 2) TLI_LAUNCH_STATS(TLI_F32, 2); else TLI_LAUNCH_STATS(TLI_F32, 1);
    } else {
        if (L.cv == 4) TLI_LAUNCH_STATS(TLI_BF16, 4); else if (L.cv == 2) TLI_LAUNCH_STATS(TLI_BF16, 2); else TLI_LAUNCH_STATS(TLI_BF16, 1);
    }
#undef TLI_LAUNCH_STATS
    return e;
}

}  // namespace

extern "C" {

int tli_create(tli_ctx **out, int device, int32_t V_t, int32_t V_d, const int32_t *id_map_host) {
    if (!out) return TLI_ERR_ARG;
    *out = nullptr;
    if (!id_map_host || device < 0) return TLI_ERR_ARG;
    if (V_t < 1 || V_d < 1) return TLI_ERR_ARG;
    if (V_t > TLI_MAX_V || V_d > TLI_MAX_V) return TLI_ERR_UNSUPPORTED;
    // host-side validation and derived tables, before any CUDA call
    std::vector<int32_t> inv(static_cast<size_t>(V_t), -1);
    const size_t mask_words = (static_cast<size_t>(V_d) + 31) / 32 + 2;
    std::vector<uint32_t> mask(mask_words, 0u);
    int32_t n_mapped = 0;
    for (int32_t x = 0; x < V_d; ++x) {
        const int32_t t = id_map_host[x];
        if (t == -1) continue;
        if (t < 0 || t >= V_t || inv[t] != -1) return TLI_ERR_BAD_MAP;
        inv[t] = x;
        mask[x >> 5] |= 1u << (x & 31);
        ++n_mapped;
    }
    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    e = cudaSetDevice(device);
    if (e != cudaSuccess) return cuda_fail(e, "cudaSetDevice");
    tli_ctx *c = new (std::nothrow) tli_ctx();
    if (!c) { cudaSetDevice(prev); return TLI_ERR_ARG; }
    c->device = device; c->V_t = V_t; c->V_d = V_d; c->n_mapped = n_mapped;
    c->d_map = nullptr; c->d_inv = nullptr; c->d_mask = nullptr; c->d_counters = nullptr; c->d_parts = nullptr;
    c->num_sms = 0;
    c->tiled = 0;
    c->max_cluster = 8; c->device_max_cluster = 8;
    c->n_shards = 1; c->shard = 0; c->wt = V_t; c->wd = V_d;
    c->t_begin = 0; c->t_count = V_t; c->d_begin = 0; c->d_count = V_d;
    int rc = TLI_OK;
    do {
        if ((e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) { rc = cuda_fail(e, "cudaDeviceGetAttribute"); break; }
        // the statistics kernel needs more dynamic shared memory than the default limit
        e = cudaSuccess;
#define TLI_SET_SMEM(DT, CV) if (e == cudaSuccess) e = cudaFuncSetAttribute(tli_stats_kernel<DT, CV>, cudaFuncAttributeMaxDynamicSharedMemorySize, kStatsSmemBytes)
        TLI_SET_SMEM(TLI_F32, 1); TLI_SET_SMEM(TLI_F32, 2); TLI_SET_SMEM(TLI_F32, 4);
        TLI_SET_SMEM(TLI_BF16, 1); TLI_SET_SMEM(TLI_BF16, 2); TLI_SET_SMEM(TLI_BF16, 4);
#undef TLI_SET_SMEM
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tli_finish_kernel<TLI_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinSmemOnePerSm);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tli_finish_kernel<TLI_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinSmemOnePerSm);
        if (e != cudaSuccess) { rc = cuda_fail(e, "cudaFuncSetAttribute"); break; }
        {
            // clusters of 16 are not portable: take them only if the driver places at least one with the
            // largest shared memory the kernel is ever given
            bool wide = true;
            for (int dt = 0; dt < 2 && wide; ++dt) {
                const void *fn = dt == 0 ? reinterpret_cast<const void *>(tli_finish_kernel<TLI_F32>)
                                         : reinterpret_cast<const void *>(tli_finish_kernel<TLI_BF16>);
                if (cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) { wide = false; break; }
                cudaLaunchConfig_t qc;
                memset(&qc, 0, sizeof qc);
                cudaLaunchAttribute qa[1];
                qa[0].id = cudaLaunchAttributeClusterDimension;
                qa[0].val.clusterDim.x = kFinMaxCluster; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
                qc.attrs = qa; qc.numAttrs = 1;
                qc.gridDim = dim3(kFinMaxCluster); qc.blockDim = dim3(kFinThreads); qc.dynamicSmemBytes = kFinSmemOnePerSm;
                int n_clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &qc) != cudaSuccess || n_clusters < 1) wide = false;
            }
            cudaGetLastError();                              // a refusal above is an answer, not an error of this call
            c->max_cluster = wide ? kFinMaxCluster : 8;
            c->device_max_cluster = c->max_cluster;
        }
        if ((e = cudaMalloc(&c->d_map, sizeof(int32_t) * V_d)) != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc map"); break; }
        if ((e = cudaMalloc(&c->d_inv, sizeof(int32_t) * (static_cast<size_t>(V_t) + 8))) != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc inverse map"); break; }
        if ((e = cudaMalloc(&c->d_mask, sizeof(uint32_t) * mask_words)) != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc mask"); break; }
        if ((e = cudaMalloc(&c->d_counters, sizeof(unsigned) * kCounterWords)) != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc counters"); break; }
        if ((e = cudaMalloc(&c->d_parts, kCtxPartsBytes)) != cudaSuccess) { rc = cuda_fail(e, "cudaMalloc partials"); break; }
        if ((e = cudaMemset(c->d_parts, 0xff, kCtxPartsBytes)) != cudaSuccess) { rc = cuda_fail(e, "cudaMemset partials"); break; }
        if ((e = cudaMemcpy(c->d_map, id_map_host, sizeof(int32_t) * V_d, cudaMemcpyHostToDevice)) != cudaSuccess) { rc = cuda_fail(e, "cudaMemcpy map"); break; }
        if ((e = cudaMemcpy(c->d_inv, inv.data(), sizeof(int32_t) * V_t, cudaMemcpyHostToDevice)) != cudaSuccess) { rc = cuda_fail(e, "cudaMemcpy inverse map"); break; }
        if ((e = cudaMemcpy(c->d_mask, mask.data(), sizeof(uint32_t) * mask_words, cudaMemcpyHostToDevice)) != cudaSuccess) { rc = cuda_fail(e, "cudaMemcpy mask"); break; }
        if ((e = cudaMemset(c->d_counters, 0, sizeof(unsigned) * kCounterWords)) != cudaSuccess) { rc = cuda_fail(e, "cudaMemset counters"); break; }
    } while (0);
    if (rc != TLI_OK) {
        cudaFree(c->d_map); cudaFree(c->d_inv); cudaFree(c->d_mask); cudaFree(c->d_counters); cudaFree(c->d_parts);
        delete c;
        cudaSetDevice(prev);
        return rc;
    }
    cudaSetDevice(prev);
    *out = c;
    return TLI_OK;
}

int tli_destroy(tli_ctx *ctx) {
    if (!ctx) return TLI_ERR_ARG;
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    cudaFree(ctx->d_map); cudaFree(ctx->d_inv); cudaFree(ctx->d_mask); cudaFree(ctx->d_counters); cudaFree(ctx->d_parts);
    if (prev >= 0) cudaSetDevice(prev);
    delete ctx;
    return TLI_OK;
}

size_t tli_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype) {
    if (!ctx || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    return make_layout(B, K, ctx->V_t, ctx->V_d, dtype, ctx->num_sms).total;
}

int tli_ctx_info(const tli_ctx *ctx, int32_t *V_t, int32_t *V_d, int32_t *n_mapped) {
    if (!ctx) return TLI_ERR_ARG;
    if (V_t) *V_t = ctx->V_t;
    if (V_d) *V_d = ctx->V_d;
    if (n_mapped) *n_mapped = ctx->n_mapped;
    return TLI_OK;
}

static int verify_impl(tli_ctx *ctx, const tli_verify_args *a, void *cuda_stream, cudaEvent_t *ev) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (ctx->n_shards != 1) return TLI_ERR_ARG;                 // a shard's context serves the tli_shard_* calls only
    if (a->B < 1 || a->K < 1) return TLI_ERR_ARG;
    if (a->B > TLI_MAX_B || a->K > TLI_MAX_K) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->target_logits || !a->drafter_logits || !a->draft_ids || !a->temperature || !a->uniforms ||
        !a->accepted || !a->next_token)
        return TLI_ERR_ARG;
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(a->target_logits) % elt || reinterpret_cast<uintptr_t>(a->drafter_logits) % elt)
        return TLI_ERR_ARG;
    if (a->t_stride_b < 0 || a->t_stride_k < 0 || a->d_stride_b < 0 || a->d_stride_k < 0) return TLI_ERR_ARG;
    Layout L = make_layout(a->B, a->K, ctx->V_t, ctx->V_d, a->dtype, ctx->num_sms, ctx->max_cluster);
    if (ctx->tiled) L.fin_cluster = 0;
    if (L.nseg >= (1ll << 32) - 4 * L.grid) return TLI_ERR_UNSUPPORTED;
    if (!a->workspace || reinterpret_cast<uintptr_t>(a->workspace) % 256 || a->workspace_bytes < L.total)
        return TLI_ERR_WORKSPACE;

    Params P;
    memset(&P, 0, sizeof P);
    P.B = a->B; P.K = a->K; P.V_t = ctx->V_t; P.V_d = ctx->V_d;
    P.zt = a->target_logits; P.t_sb = a->t_stride_b; P.t_sk = a->t_stride_k;
    P.zd = a->drafter_logits; P.d_sb = a->d_stride_b; P.d_sk = a->d_stride_k;
    P.map = ctx->d_map; P.inv = ctx->d_inv; P.maskbits = ctx->d_mask; P.n_mapped = ctx->n_mapped;
    P.draft = a->draft_ids; P.tau = a->temperature; P.u = a->uniforms;
    P.draft_len = a->draft_lengths;
    P.accepted = a->accepted; P.next_token = a->next_token; P.status = a->row_status;
    P.p_out = a->p_draft; P.q_out = a->q_draft;
    char *ws = reinterpret_cast<char *>(a->workspace);
    P.part_t = reinterpret_cast<float2 *>(ws + L.part_t);
    P.part_d = reinterpret_cast<float2 *>(ws + L.part_d);
    P.sel = reinterpret_cast<RowSel *>(ws + L.sel);
    P.tilesum = reinterpret_cast<double *>(ws + L.tilesum);
    P.cnt_stats = ctx->d_counters;
    P.cnt_sample = ctx->d_counters + (TLI_MAX_B + 1);
    P.error = ctx->d_counters + 3 * (TLI_MAX_B + 1);
    P.seg_counter = reinterpret_cast<unsigned long long *>(P.error + 4); P.cta_done = P.error + 2;
    // many tiles: a fence and a ticket per tile CTA cost more than one more small kernel
    P.split_select = (static_cast<long long>(a->B) * L.ntile >= 4096) ? 1 : 0;
    P.ntile = L.ntile;
    P.fin_slice = L.fin_slice; P.fin_dvec = L.fin_dvec;
    {
        // cluster form: partials in the context's own buffer, where "not yet stored" can be told from the data
        const size_t n_t = static_cast<size_t>(a->B) * (a->K + 1) * L.nst, n_d = static_cast<size_t>(a->B) * a->K * L.nsd;
        if (L.fin_cluster && (n_t + n_d) * sizeof(float2) <= kCtxPartsBytes) {
            P.part_t = ctx->d_parts;
            P.part_d = ctx->d_parts + n_t;
            P.poll_parts = 1;
            P.early_trigger = L.grid < static_cast<unsigned>(kCtasPerSm * ctx->num_sms) ? 1 : 0;
        }
    }
    P.seg_vec = L.seg_vec; P.nst = L.nst; P.nsd = L.nsd;
    P.div_per_b = make_fast_div(static_cast<unsigned>((P.K + 1) * L.nst + P.K * L.nsd));
    P.div_nst = make_fast_div(static_cast<unsigned>(L.nst)); P.div_nsd = make_fast_div(static_cast<unsigned>(L.nsd));

    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (ev) cudaEventRecord(ev[0], stream);
    const dim3 grid2(static_cast<unsigned>(L.ntile), static_cast<unsigned>(a->B));
    cudaError_t e = launch_stats(P, L, a->dtype, stream);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_stats_kernel");
    if (ev) cudaEventRecord(ev[1], stream);

    // The kernels after the first are launched as programmatic dependents: no predecessor triggers
    // early, so they still start only when it is done, but their launch is set up while it runs
    // (4-6 us per call).  Each begins with griddepcontrol.wait.
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1; cfg.stream = stream;
    if (L.fin_cluster) {
        // decision and extra token by one cluster per sequence
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = static_cast<unsigned>(L.fin_cluster);
        attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
        cfg.blockDim = dim3(kFinThreads); cfg.dynamicSmemBytes = L.fin_smem;
        cfg.gridDim = dim3(static_cast<unsigned>(L.fin_cluster), static_cast<unsigned>(a->B));
        if (ev) cudaEventRecord(ev[2], stream);
        if (a->dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_finish_kernel<TLI_F32>, P);
        else e = cudaLaunchKernelEx(&cfg, tli_finish_kernel<TLI_BF16>, P);
        if (e != cudaSuccess) return cuda_fail(e, "launch tli_finish_kernel");
        if (ev) cudaEventRecord(ev[3], stream);
        return TLI_OK;
    }
    cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = 0;
    cfg.gridDim = dim3(static_cast<unsigned>(a->B));
    if (a->dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_decide_kernel<TLI_F32>, P);
    else e = cudaLaunchKernelEx(&cfg, tli_decide_kernel<TLI_BF16>, P);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_decide_kernel");
    if (ev) cudaEventRecord(ev[2], stream);
    cfg.gridDim = grid2;
    if (a->dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_sample_kernel<TLI_F32>, P);
    else e = cudaLaunchKernelEx(&cfg, tli_sample_kernel<TLI_BF16>, P);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_sample_kernel");
    if (P.split_select) {
        cfg.gridDim = dim3(static_cast<unsigned>(a->B));
        if (a->dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_select_kernel<TLI_F32>, P);
        else e = cudaLaunchKernelEx(&cfg, tli_select_kernel<TLI_BF16>, P);
        if (e != cudaSuccess) return cuda_fail(e, "launch tli_select_kernel");
    }
    if (ev) cudaEventRecord(ev[3], stream);
    return TLI_OK;
}

int tli_verify(tli_ctx *ctx, const tli_verify_args *a, void *cuda_stream) {
    return verify_impl(ctx, a, cuda_stream, nullptr);
}

size_t tli_draft_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t R, int32_t dtype) {
    if (!ctx || B < 1 || R < 1 || static_cast<long long>(B) * R > TLI_MAX_B) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    const size_t nstrip = static_cast<size_t>(chunks_per_row(ctx->V_d, dtype, kVecPerTile)) * kStripsPerTile;
    return align_up(sizeof(DraftPart) * static_cast<size_t>(B) * R * nstrip, 256);
}

// The sampling kernels on `rows` = B * R rows: tiles, then (large batches) the selections.
static int launch_row_sampler(DraftParams &P, int dtype, cudaStream_t stream) {
    const int rows = P.B * P.R;
    P.ntile = chunks_per_row(P.V_d, dtype, kVecPerTile);
    P.nstrip = P.ntile * kStripsPerTile;
    // many tiles: a fence and a ticket per tile CTA cost more than one more small kernel
    P.split = (static_cast<long long>(rows) * P.ntile >= 4096) ? 1 : 0;
    const dim3 grid(static_cast<unsigned>(P.ntile), static_cast<unsigned>(rows));
    if (dtype == TLI_F32) tli_draft_kernel<TLI_F32><<<grid, kThreads, 0, stream>>>(P);
    else tli_draft_kernel<TLI_BF16><<<grid, kThreads, 0, stream>>>(P);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_draft_kernel");
    if (P.split) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.gridDim = dim3(static_cast<unsigned>(rows)); cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = 0; cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = 1;
        if (dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_draft_select_kernel<TLI_F32>, P);
        else e = cudaLaunchKernelEx(&cfg, tli_draft_select_kernel<TLI_BF16>, P);
        if (e != cudaSuccess) return cuda_fail(e, "launch tli_draft_select_kernel");
    }
    return TLI_OK;
}

int tli_draft_sample(tli_ctx *ctx, const tli_draft_args *a, void *cuda_stream) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->R < 1) return TLI_ERR_ARG;
    if (static_cast<long long>(a->B) * a->R > TLI_MAX_B) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->drafter_logits || !a->temperature || !a->uniforms || !a->draft_ids) return TLI_ERR_ARG;
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(a->drafter_logits) % elt) return TLI_ERR_ARG;
    if (a->d_stride_b < 0 || a->d_stride_r < 0) return TLI_ERR_ARG;
    const size_t need = tli_draft_workspace_bytes(ctx, a->B, a->R, a->dtype);
    if (!a->workspace || reinterpret_cast<uintptr_t>(a->workspace) % 256 || a->workspace_bytes < need)
        return TLI_ERR_WORKSPACE;
    DraftParams P;
    P.B = a->B; P.R = a->R; P.V_d = ctx->V_d;
    P.zd = a->drafter_logits; P.d_sb = a->d_stride_b; P.d_sr = a->d_stride_r;
    P.maskbits = ctx->d_mask; P.lengths = nullptr; P.tau = a->temperature; P.u = a->uniforms;
    P.draft_ids = a->draft_ids; P.q_out = a->q_draft; P.status = a->draft_status;
    P.part = reinterpret_cast<DraftPart *>(a->workspace);
    P.cnt = ctx->d_counters + (TLI_MAX_B + 1);           // the sampling pass's tickets: zero between calls
    return launch_row_sampler(P, a->dtype, reinterpret_cast<cudaStream_t>(cuda_stream));
}

namespace {
struct SlemLayout { size_t part, sampled, flags, total; };
SlemLayout slem_layout(int B, int M, int V_t, int dtype) {
    SlemLayout L;
    const size_t rows = static_cast<size_t>(B) * (M + 1);
    const size_t nstrip = static_cast<size_t>(chunks_per_row(V_t, dtype, kVecPerTile)) * kStripsPerTile;
    size_t off = 0;
    L.part = off;    off = align_up(off + sizeof(DraftPart) * rows * nstrip, 256);
    L.sampled = off; off = align_up(off + sizeof(int) * rows, 256);
    L.flags = off;   off = align_up(off + sizeof(int) * rows, 256);
    L.total = off;
    return L;
}
}  // namespace

size_t tli_slem_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t M, int32_t dtype) {
    if (!ctx || B < 1 || M < 0 || M > TLI_MAX_K || static_cast<long long>(B) * (M + 1) > TLI_MAX_B) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    return slem_layout(B, M, ctx->V_t, dtype).total;
}

int tli_slem_verify(tli_ctx *ctx, const tli_slem_args *a, void *cuda_stream) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->M < 0) return TLI_ERR_ARG;
    if (a->M > TLI_MAX_K || static_cast<long long>(a->B) * (a->M + 1) > TLI_MAX_B) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->target_logits || !a->temperature || !a->uniforms || !a->accepted || !a->next_token) return TLI_ERR_ARG;
    if (a->M > 0 && !a->candidates) return TLI_ERR_ARG;
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(a->target_logits) % elt) return TLI_ERR_ARG;
    if (a->t_stride_b < 0 || a->t_stride_k < 0) return TLI_ERR_ARG;
    const SlemLayout L = slem_layout(a->B, a->M, ctx->V_t, a->dtype);
    if (!a->workspace || reinterpret_cast<uintptr_t>(a->workspace) % 256 || a->workspace_bytes < L.total)
        return TLI_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(a->workspace);
    int *sampled = a->sampled ? a->sampled : reinterpret_cast<int *>(ws + L.sampled);
    int *flags = reinterpret_cast<int *>(ws + L.flags);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    DraftParams P;
    P.B = a->B; P.R = a->M + 1; P.V_d = ctx->V_t;
    P.zd = a->target_logits; P.d_sb = a->t_stride_b; P.d_sr = a->t_stride_k;
    P.maskbits = nullptr; P.lengths = a->lengths; P.tau = a->temperature; P.u = a->uniforms;
    P.draft_ids = sampled; P.q_out = nullptr; P.status = flags;
    P.part = reinterpret_cast<DraftPart *>(ws + L.part);
    P.cnt = ctx->d_counters + (TLI_MAX_B + 1);
    const int rc = launch_row_sampler(P, a->dtype, stream);
    if (rc != TLI_OK) return rc;
    SlemParams Q;
    Q.B = a->B; Q.M = a->M; Q.candidates = a->candidates; Q.lengths = a->lengths; Q.tau = a->temperature;
    Q.sampled = sampled; Q.row_flags = flags;
    Q.accepted = a->accepted; Q.next_token = a->next_token; Q.status = a->row_status;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(static_cast<unsigned>((a->B + 127) / 128)); cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = 0; cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, tli_slem_match_kernel, Q);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_slem_match_kernel");
    return TLI_OK;
}

// ---- vocabulary-sharded verification ----

namespace {

struct ShardLayout { Layout L; size_t tilesum_p, total; int row_pitch; };

ShardLayout make_shard_layout(const tli_ctx *ctx, int B, int K, int dtype) {
    ShardLayout SL;
    SL.L = make_layout(B, K, ctx->t_count, ctx->d_count, dtype, ctx->num_sms);
    SL.tilesum_p = SL.L.total;
    SL.total = align_up(SL.tilesum_p + sizeof(double) * static_cast<size_t>(B) * SL.L.ntile, 256);
    const int epv = dtype == TLI_F32 ? 4 : 8;
    SL.row_pitch = (ctx->wd + epv - 1) / epv * epv;
    return SL;
}

// Argument checks and kernel parameters shared by the four sharded calls.
int shard_params(tli_ctx *ctx, const tli_verify_args *a, ShardParams &S, ShardLayout &SL) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->K < 1) return TLI_ERR_ARG;
    if (a->B > TLI_MAX_B || a->K > TLI_MAX_K) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->target_logits || !a->drafter_logits || !a->draft_ids || !a->temperature || !a->uniforms ||
        !a->accepted || !a->next_token)
        return TLI_ERR_ARG;
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(a->target_logits) % elt || reinterpret_cast<uintptr_t>(a->drafter_logits) % elt)
        return TLI_ERR_ARG;
    if (a->t_stride_b < 0 || a->t_stride_k < 0 || a->d_stride_b < 0 || a->d_stride_k < 0) return TLI_ERR_ARG;
    if (a->draft_lengths) return TLI_ERR_UNSUPPORTED;
    SL = make_shard_layout(ctx, a->B, a->K, a->dtype);
    if (SL.L.nseg >= (1ll << 32) - 4 * SL.L.grid) return TLI_ERR_UNSUPPORTED;
    if (!a->workspace || reinterpret_cast<uintptr_t>(a->workspace) % 256 || a->workspace_bytes < SL.total)
        return TLI_ERR_WORKSPACE;
    memset(&S, 0, sizeof S);
    Params &P = S.P;
    const Layout &L = SL.L;
    P.B = a->B; P.K = a->K; P.V_t = ctx->t_count; P.V_d = ctx->d_count;
    P.zt = a->target_logits; P.t_sb = a->t_stride_b; P.t_sk = a->t_stride_k;
    P.zd = a->drafter_logits; P.d_sb = a->d_stride_b; P.d_sk = a->d_stride_k;
    P.map = ctx->d_map; P.inv = ctx->d_inv; P.maskbits = ctx->d_mask; P.n_mapped = ctx->n_mapped;
    P.draft = a->draft_ids; P.tau = a->temperature; P.u = a->uniforms;
    P.accepted = a->accepted; P.next_token = a->next_token; P.status = a->row_status;
    P.p_out = a->p_draft; P.q_out = a->q_draft;
    char *ws = reinterpret_cast<char *>(a->workspace);
    P.part_t = reinterpret_cast<float2 *>(ws + L.part_t);
    P.part_d = reinterpret_cast<float2 *>(ws + L.part_d);
    P.sel = reinterpret_cast<RowSel *>(ws + L.sel);
    P.tilesum = reinterpret_cast<double *>(ws + L.tilesum);
    P.tilesum_p = reinterpret_cast<double *>(ws + SL.tilesum_p);
    P.cnt_stats = ctx->d_counters;
    P.cnt_sample = ctx->d_counters + (TLI_MAX_B + 1);
    P.error = ctx->d_counters + 3 * (TLI_MAX_B + 1);
    P.seg_counter = reinterpret_cast<unsigned long long *>(P.error + 4); P.cta_done = P.error + 2;
    P.ntile = L.ntile;
    P.seg_vec = L.seg_vec; P.nst = L.nst; P.nsd = L.nsd;
    P.div_per_b = make_fast_div(static_cast<unsigned>((P.K + 1) * L.nst + P.K * L.nsd));
    P.div_nst = make_fast_div(static_cast<unsigned>(L.nst)); P.div_nsd = make_fast_div(static_cast<unsigned>(L.nsd));
    P.t_begin = ctx->t_begin; P.d_begin = ctx->d_begin;
    P.sh_wd = ctx->wd; P.sh_stride = static_cast<long long>(a->B) * SL.row_pitch;
    S.G = ctx->n_shards; S.g = ctx->shard; S.wt = ctx->wt; S.wd = ctx->wd;
    S.V_t_all = ctx->V_t; S.V_d_all = ctx->V_d;
    S.row_pitch = SL.row_pitch;
    return TLI_OK;
}

}  // namespace

int tli_shard_create(tli_ctx **out, int device, int32_t V_t, int32_t V_d, const int32_t *id_map_host,
                     int32_t n_shards, int32_t shard) {
    if (out) *out = nullptr;
    if (n_shards < 1 || n_shards > TLI_MAX_SHARDS || shard < 0 || shard >= n_shards) return TLI_ERR_ARG;
    const int rc = tli_create(out, device, V_t, V_d, id_map_host);
    if (rc != TLI_OK) return rc;
    tli_ctx *c = *out;
    c->n_shards = n_shards; c->shard = shard;
    c->wt = (V_t + n_shards - 1) / n_shards;
    c->wd = (V_d + n_shards - 1) / n_shards;
    auto clip = [](long long x, int32_t hi) { return static_cast<int32_t>(x < hi ? x : hi); };
    c->t_begin = clip(static_cast<long long>(shard) * c->wt, V_t);
    c->t_count = clip(static_cast<long long>(shard + 1) * c->wt, V_t) - c->t_begin;
    c->d_begin = clip(static_cast<long long>(shard) * c->wd, V_d);
    c->d_count = clip(static_cast<long long>(shard + 1) * c->wd, V_d) - c->d_begin;
    return TLI_OK;
}

int tli_shard_info(const tli_ctx *ctx, int32_t *t_begin, int32_t *t_count, int32_t *d_begin, int32_t *d_count,
                   int32_t *t_width, int32_t *d_width) {
    if (!ctx) return TLI_ERR_ARG;
    if (t_begin) *t_begin = ctx->t_begin;
    if (t_count) *t_count = ctx->t_count;
    if (d_begin) *d_begin = ctx->d_begin;
    if (d_count) *d_count = ctx->d_count;
    if (t_width) *t_width = ctx->wt;
    if (d_width) *d_width = ctx->wd;
    return TLI_OK;
}

size_t tli_shard_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype) {
    if (!ctx || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    return make_shard_layout(ctx, B, K, dtype).total;
}

size_t tli_shard_record_bytes(const tli_ctx *ctx, int32_t B, int32_t K) {
    if (!ctx || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return 0;
    return sizeof(double) * static_cast<size_t>(B) * shard_record_len(K);
}

size_t tli_shard_rows_bytes(const tli_ctx *ctx, int32_t B, int32_t dtype) {
    if (!ctx || B < 1 || B > TLI_MAX_B || (dtype != TLI_F32 && dtype != TLI_BF16)) return 0;
    const size_t epv = dtype == TLI_F32 ? 4 : 8;
    return static_cast<size_t>(B) * ((ctx->wd + epv - 1) / epv) * 16;
}

int tli_shard_stats(tli_ctx *ctx, const tli_verify_args *a, void *record_out, void *cuda_stream) {
    ShardParams S; ShardLayout SL;
    const int rc = shard_params(ctx, a, S, SL);
    if (rc != TLI_OK) return rc;
    if (!record_out || reinterpret_cast<uintptr_t>(record_out) % 8) return TLI_ERR_ARG;
    S.record = reinterpret_cast<double *>(record_out);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = launch_stats(S.P, SL.L, a->dtype, stream);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_stats_kernel");
    if (a->dtype == TLI_F32) tli_shard_fold_kernel<TLI_F32><<<a->B, kThreads, 0, stream>>>(S);
    else tli_shard_fold_kernel<TLI_BF16><<<a->B, kThreads, 0, stream>>>(S);
    e = cudaGetLastError();
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "launch tli_shard_fold_kernel");
}

int tli_shard_decide(tli_ctx *ctx, const tli_verify_args *a, const void *records_all, void *rows_out, void *cuda_stream) {
    ShardParams S; ShardLayout SL;
    const int rc = shard_params(ctx, a, S, SL);
    if (rc != TLI_OK) return rc;
    if (!records_all || !rows_out || reinterpret_cast<uintptr_t>(records_all) % 8 || reinterpret_cast<uintptr_t>(rows_out) % 16)
        return TLI_ERR_ARG;
    S.records = reinterpret_cast<const double *>(records_all);
    S.rows_out = rows_out;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    tli_shard_decide_kernel<<<a->B, 128, 0, stream>>>(S);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_shard_decide_kernel");
    const int epv = a->dtype == TLI_F32 ? 4 : 8;
    const dim3 grid(static_cast<unsigned>((SL.row_pitch / epv + kThreads - 1) / kThreads), static_cast<unsigned>(a->B));
    if (a->dtype == TLI_F32) tli_shard_pack_kernel<TLI_F32><<<grid, kThreads, 0, stream>>>(S);
    else tli_shard_pack_kernel<TLI_BF16><<<grid, kThreads, 0, stream>>>(S);
    e = cudaGetLastError();
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "launch tli_shard_pack_kernel");
}

int tli_shard_weights(tli_ctx *ctx, const tli_verify_args *a, const void *rows_all, void *mass_out, void *cuda_stream) {
    ShardParams S; ShardLayout SL;
    const int rc = shard_params(ctx, a, S, SL);
    if (rc != TLI_OK) return rc;
    if (!rows_all || !mass_out || reinterpret_cast<uintptr_t>(rows_all) % 16 || reinterpret_cast<uintptr_t>(mass_out) % 8)
        return TLI_ERR_ARG;
    S.rows_all = rows_all;
    S.mass = reinterpret_cast<double *>(mass_out);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const dim3 grid(static_cast<unsigned>(SL.L.ntile), static_cast<unsigned>(a->B));
    if (a->dtype == TLI_F32) tli_shard_weights_kernel<TLI_F32><<<grid, kThreads, 0, stream>>>(S);
    else tli_shard_weights_kernel<TLI_BF16><<<grid, kThreads, 0, stream>>>(S);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_shard_weights_kernel");
    tli_shard_mass_kernel<<<(a->B + 127) / 128, 128, 0, stream>>>(S);
    e = cudaGetLastError();
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "launch tli_shard_mass_kernel");
}

int tli_shard_select(tli_ctx *ctx, const tli_verify_args *a, const void *rows_all, const void *masses_all, void *cuda_stream) {
    ShardParams S; ShardLayout SL;
    const int rc = shard_params(ctx, a, S, SL);
    if (rc != TLI_OK) return rc;
    if (!rows_all || !masses_all || reinterpret_cast<uintptr_t>(rows_all) % 16 || reinterpret_cast<uintptr_t>(masses_all) % 8)
        return TLI_ERR_ARG;
    S.rows_all = rows_all;
    S.masses = reinterpret_cast<const double *>(masses_all);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (a->dtype == TLI_F32) tli_shard_select_kernel<TLI_F32><<<a->B, kThreads, 0, stream>>>(S);
    else tli_shard_select_kernel<TLI_BF16><<<a->B, kThreads, 0, stream>>>(S);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "launch tli_shard_select_kernel");
}

int tli_selftest_bounded_wait(tli_ctx *ctx, void *cuda_stream, unsigned polls, int *gave_up) {
    if (!ctx || !gave_up || polls == 0 || polls > kWaitLimit) return TLI_ERR_ARG;
    // scratch: the two unused words after the schedulers' counters, so the sticky error word stays clean
    int *d_result = reinterpret_cast<int *>(ctx->d_counters + 3 * (TLI_MAX_B + 1) + 4);
    unsigned *d_err = ctx->d_counters + 3 * (TLI_MAX_B + 1) + 6;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(d_result, 0, 3 * sizeof(int), stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    tli_bounded_wait_kernel<<<1, 32, 0, stream>>>(polls, d_result, d_err);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "launch tli_bounded_wait_kernel");
    int h[3] = {0, 0, 0};
    if ((e = cudaMemcpyAsync(h, d_result, sizeof h, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    *gave_up = (h[0] == 1 && h[1] == 1) ? 1 : 0;
    return TLI_OK;
}

int tli_reset(tli_ctx *ctx, void *cuda_stream) {
    if (!ctx) return TLI_ERR_ARG;
    cudaError_t e = cudaMemsetAsync(ctx->d_counters, 0, sizeof(unsigned) * kCounterWords, reinterpret_cast<cudaStream_t>(cuda_stream));
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_parts, 0xff, kCtxPartsBytes, reinterpret_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "cudaMemsetAsync counters");
}

int tli_set_tiled(tli_ctx *ctx, int enabled) {
    if (!ctx) return TLI_ERR_ARG;
    ctx->tiled = enabled ? 1 : 0;
    return TLI_OK;
}

int tli_set_max_cluster(tli_ctx *ctx, int ctas) {
    if (!ctx || (ctas != 8 && ctas != kFinMaxCluster)) return TLI_ERR_ARG;
    if (ctas > ctx->device_max_cluster) return TLI_ERR_UNSUPPORTED;
    ctx->max_cluster = ctas;
    return TLI_OK;
}

int tli_verify_plan(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype, int32_t *plan) {
    if (!ctx || !plan || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return TLI_ERR_ARG;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return TLI_ERR_ARG;
    Layout L = make_layout(B, K, ctx->t_count, ctx->d_count, dtype, ctx->num_sms, ctx->max_cluster);
    if (ctx->tiled || ctx->n_shards != 1) L.fin_cluster = 0;
    const int split = (static_cast<long long>(B) * L.ntile >= 4096) ? 1 : 0;
    plan[0] = L.fin_cluster ? 2 : 3 + split;         // kernel launches per call
    plan[1] = L.fin_cluster;                         // CTAs per sequence of the cluster kernel, 0: tile kernels
    plan[2] = static_cast<int32_t>(L.grid);          // CTAs of the statistics kernel
    plan[3] = L.cv * kSThreads * 16;                 // bytes per stage
    plan[4] = L.seg_vec * 16;                        // bytes per segment
    plan[5] = L.nst; plan[6] = L.nsd;                // segments per target / drafter row
    plan[7] = static_cast<int32_t>(L.fin_smem);      // shared memory of a cluster CTA
    return TLI_OK;
}

int tli_launch_probe(tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype, void *cuda_stream) {
    if (!ctx || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return TLI_ERR_ARG;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return TLI_ERR_ARG;
    Layout L = make_layout(B, K, ctx->V_t, ctx->V_d, dtype, ctx->num_sms, ctx->max_cluster);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    static std::once_flag once;
    std::call_once(once, [] {
        cudaFuncSetAttribute(tli_probe_first_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStatsSmemBytes);
        cudaFuncSetAttribute(tli_probe_second_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kFinSmemOnePerSm));
        cudaFuncSetAttribute(tli_probe_second_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    });
    tli_probe_first_kernel<<<L.grid, kSThreads + 32, kStatsSmemBytes, stream>>>(0);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_probe_first_kernel");
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    const int C = L.fin_cluster ? L.fin_cluster : 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(C); attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2; cfg.stream = stream;
    cfg.blockDim = dim3(kFinThreads); cfg.dynamicSmemBytes = L.fin_cluster ? L.fin_smem : 0;
    cfg.gridDim = dim3(static_cast<unsigned>(C), static_cast<unsigned>(B));
    e = cudaLaunchKernelEx(&cfg, tli_probe_second_kernel, 0);
    return e == cudaSuccess ? TLI_OK : cuda_fail(e, "launch tli_probe_second_kernel");
}

int tli_verify_profile(tli_ctx *ctx, const tli_verify_args *a, void *cuda_stream, float *ms) {
    if (!ms) return TLI_ERR_ARG;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < 4 && e == cudaSuccess; ++i) e = cudaEventCreate(&ev[i]);
    int rc = (e == cudaSuccess) ? verify_impl(ctx, a, cuda_stream, ev) : cuda_fail(e, "cudaEventCreate");
    if (rc == TLI_OK) {
        if ((e = cudaEventSynchronize(ev[3])) != cudaSuccess) rc = cuda_fail(e, "cudaEventSynchronize");
        else for (int i = 0; i < 3; ++i) cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1]);
    }
    for (int i = 0; i < 4; ++i) if (ev[i]) cudaEventDestroy(ev[i]);
    return rc;
}

// ---------------------------------------------------------------------------
// tli_verify_static: the same verification with library-resident scratch
// ---------------------------------------------------------------------------

// Scratch for callers that cannot allocate.  It lives in the library's device image: every GPU
// that loads the library carries these bytes until the process exits, whether or not it is used.
static __device__ __align__(256) unsigned char g_static_scratch[TLI_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void *g_static_scratch_ptr[kMaxDevices];       // device address of g_static_scratch, per device
bool g_static_scratch_ready[kMaxDevices];
std::mutex g_static_scratch_mutex;

// In host code the name g_static_scratch is only a handle for the runtime, not an address a
// kernel could use; the device address has to be asked for, once per device, with that device current.
int static_scratch_address(int device, void **out) {
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ready[device]) {
        void *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(g_static_scratch)");
        if (!ptr) return cuda_fail(cudaErrorInvalidSymbol, "cudaGetSymbolAddress(g_static_scratch)");
        g_static_scratch_ptr[device] = ptr;
        g_static_scratch_ready[device] = true;
    }
    *out = g_static_scratch_ptr[device];
    return TLI_OK;
}
}  // namespace

int tli_verify_static(tli_ctx *ctx, const tli_verify_args *a, void *cuda_stream) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->K < 1) return TLI_ERR_ARG;
    if (a->B > TLI_MAX_B || a->K > TLI_MAX_K) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (make_layout(a->B, a->K, ctx->V_t, ctx->V_d, a->dtype, ctx->num_sms).total > TLI_STATIC_SCRATCH_BYTES)
        return TLI_ERR_STATIC_SCRATCH;
    int device = -1;
    const cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (device != ctx->device || device < 0 || device >= kMaxDevices) return TLI_ERR_ARG;
    void *scratch = nullptr;
    const int rc = static_scratch_address(device, &scratch);
    if (rc != TLI_OK) return rc;
    tli_verify_args b = *a;
    b.workspace = scratch;
    b.workspace_bytes = TLI_STATIC_SCRATCH_BYTES;
    return verify_impl(ctx, &b, cuda_stream, nullptr);
}

namespace {
struct RateLayout { size_t strips, rows, tiles, total; int nstrip_t, nstrip_d, nstrip_max, ntile_t, ntile_d; };
RateLayout rate_layout(const tli_ctx *ctx, int B, int K, int dtype) {
    RateLayout L;
    L.ntile_t = chunks_per_row(ctx->V_t, dtype, kVecPerTile);
    L.ntile_d = chunks_per_row(ctx->V_d, dtype, kVecPerTile);
    L.nstrip_t = L.ntile_t * kStripsPerTile; L.nstrip_d = L.ntile_d * kStripsPerTile;
    L.nstrip_max = L.nstrip_t > L.nstrip_d ? L.nstrip_t : L.nstrip_d;
    const size_t bk = static_cast<size_t>(B) * K;
    size_t off = 0;
    L.strips = off; off = align_up(off + sizeof(RateStrip) * 2 * bk * L.nstrip_max, 256);
    L.rows = off;   off = align_up(off + sizeof(RateRow) * 2 * bk, 256);
    L.tiles = off;  off = align_up(off + sizeof(double2) * bk * L.ntile_d, 256);
    L.total = off;
    return L;
}
}  // namespace

size_t tli_rates_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype) {
    if (!ctx || B < 1 || K < 1 || K > TLI_MAX_K || 2ll * B * K > TLI_MAX_B) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    return rate_layout(ctx, B, K, dtype).total;
}

int tli_acceptance_rates(tli_ctx *ctx, const tli_rates_args *a, void *cuda_stream) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->K < 1) return TLI_ERR_ARG;
    if (a->K > TLI_MAX_K || 2ll * a->B * a->K > TLI_MAX_B) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->target_logits || !a->drafter_logits || !a->temperature || !a->mass || !a->alpha_union || !a->alpha_tli)
        return TLI_ERR_ARG;
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(a->target_logits) % elt || reinterpret_cast<uintptr_t>(a->drafter_logits) % elt)
        return TLI_ERR_ARG;
    if (a->t_stride_b < 0 || a->t_stride_k < 0 || a->d_stride_b < 0 || a->d_stride_k < 0) return TLI_ERR_ARG;
    const RateLayout L = rate_layout(ctx, a->B, a->K, a->dtype);
    if (!a->workspace || reinterpret_cast<uintptr_t>(a->workspace) % 256 || a->workspace_bytes < L.total)
        return TLI_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(a->workspace);
    RateParams P;
    P.B = a->B; P.K = a->K; P.V_t = ctx->V_t; P.V_d = ctx->V_d;
    P.zt = a->target_logits; P.t_sb = a->t_stride_b; P.t_sk = a->t_stride_k;
    P.zd = a->drafter_logits; P.d_sb = a->d_stride_b; P.d_sk = a->d_stride_k;
    P.map = ctx->d_map; P.maskbits = ctx->d_mask; P.tau = a->temperature;
    P.mass = a->mass; P.alpha_union = a->alpha_union; P.alpha_tli = a->alpha_tli; P.status = a->position_status;
    P.strips = reinterpret_cast<RateStrip *>(ws + L.strips);
    P.rows = reinterpret_cast<RateRow *>(ws + L.rows);
    P.tiles = reinterpret_cast<double2 *>(ws + L.tiles);
    P.cnt = ctx->d_counters + (TLI_MAX_B + 1);
    P.nstrip_t = L.nstrip_t; P.nstrip_d = L.nstrip_d; P.nstrip_max = L.nstrip_max; P.ntile_d = L.ntile_d;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const int bk = a->B * a->K;
    const dim3 g1(static_cast<unsigned>(L.ntile_t > L.ntile_d ? L.ntile_t : L.ntile_d), static_cast<unsigned>(2 * bk));
    if (a->dtype == TLI_F32) tli_rate_stats_kernel<TLI_F32><<<g1, kThreads, 0, stream>>>(P);
    else tli_rate_stats_kernel<TLI_BF16><<<g1, kThreads, 0, stream>>>(P);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_rate_stats_kernel");
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1; cfg.stream = stream; cfg.dynamicSmemBytes = 0;
    cfg.gridDim = dim3(static_cast<unsigned>(2 * bk)); cfg.blockDim = dim3(128);
    if ((e = cudaLaunchKernelEx(&cfg, tli_rate_rows_kernel, P)) != cudaSuccess) return cuda_fail(e, "launch tli_rate_rows_kernel");
    cfg.gridDim = dim3(static_cast<unsigned>(L.ntile_d), static_cast<unsigned>(bk)); cfg.blockDim = dim3(kThreads);
    if (a->dtype == TLI_F32) e = cudaLaunchKernelEx(&cfg, tli_rate_pairs_kernel<TLI_F32>, P);
    else e = cudaLaunchKernelEx(&cfg, tli_rate_pairs_kernel<TLI_BF16>, P);
    if (e != cudaSuccess) return cuda_fail(e, "launch tli_rate_pairs_kernel");
    return TLI_OK;
}

namespace {
struct HostLayout { size_t zt, zd, draft, tau, u, out, status, ws, total; };
HostLayout host_layout(const tli_ctx *ctx, int B, int K, int dtype) {
    HostLayout L;
    const size_t elt = dtype == TLI_F32 ? 4 : 2;
    size_t off = 0;
    L.zt = off;     off = align_up(off + elt * static_cast<size_t>(B) * (K + 1) * ctx->V_t, 256);
    L.zd = off;     off = align_up(off + elt * static_cast<size_t>(B) * K * ctx->V_d, 256);
    L.draft = off;  off = align_up(off + sizeof(int) * static_cast<size_t>(B) * K, 256);
    L.tau = off;    off = align_up(off + sizeof(float) * static_cast<size_t>(B), 256);
    L.u = off;      off = align_up(off + sizeof(float) * static_cast<size_t>(B) * (K + 1), 256);
    L.out = off;    off = align_up(off + sizeof(int) * 2 * static_cast<size_t>(B), 256);     // accepted, next_token
    L.status = off; off = align_up(off + sizeof(int) * static_cast<size_t>(B), 256);
    L.ws = off;     off = align_up(off + make_layout(B, K, ctx->V_t, ctx->V_d, dtype, ctx->num_sms).total, 256);
    L.total = off;
    return L;
}
}  // namespace

size_t tli_verify_host_buffer_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype) {
    if (!ctx || B < 1 || K < 1 || B > TLI_MAX_B || K > TLI_MAX_K) return 0;
    if (dtype != TLI_F32 && dtype != TLI_BF16) return 0;
    return host_layout(ctx, B, K, dtype).total;
}

int tli_verify_host(tli_ctx *ctx, const tli_verify_host_args *a, void *cuda_stream) {
    if (!ctx || !a) return TLI_ERR_ARG;
    if (a->B < 1 || a->K < 1) return TLI_ERR_ARG;
    if (a->B > TLI_MAX_B || a->K > TLI_MAX_K) return TLI_ERR_UNSUPPORTED;
    if (a->dtype != TLI_F32 && a->dtype != TLI_BF16) return TLI_ERR_ARG;
    if (!a->target_logits || !a->drafter_logits || !a->draft_ids || !a->temperature || !a->uniforms ||
        !a->accepted || !a->next_token)
        return TLI_ERR_ARG;
    const HostLayout L = host_layout(ctx, a->B, a->K, a->dtype);
    if (!a->device_buffer || reinterpret_cast<uintptr_t>(a->device_buffer) % 256 || a->device_buffer_bytes < L.total)
        return TLI_ERR_WORKSPACE;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    char *d = reinterpret_cast<char *>(a->device_buffer);
    const size_t elt = a->dtype == TLI_F32 ? 4 : 2;
    const size_t B = static_cast<size_t>(a->B), K = static_cast<size_t>(a->K);
    struct { size_t off; const void *src; size_t bytes; } in[5] = {
        {L.zt, a->target_logits, elt * B * (K + 1) * ctx->V_t},
        {L.zd, a->drafter_logits, elt * B * K * ctx->V_d},
        {L.draft, a->draft_ids, sizeof(int) * B * K},
        {L.tau, a->temperature, sizeof(float) * B},
        {L.u, a->uniforms, sizeof(float) * B * (K + 1)},
    };
    cudaError_t e;
    for (int i = 0; i < 5; ++i)
        if ((e = cudaMemcpyAsync(d + in[i].off, in[i].src, in[i].bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
            return cuda_fail(e, "cudaMemcpyAsync to the device");
    tli_verify_args v;
    memset(&v, 0, sizeof v);
    v.B = a->B; v.K = a->K; v.dtype = a->dtype;
    v.target_logits = d + L.zt; v.t_stride_b = static_cast<int64_t>(K + 1) * ctx->V_t; v.t_stride_k = ctx->V_t;
    v.drafter_logits = d + L.zd; v.d_stride_b = static_cast<int64_t>(K) * ctx->V_d; v.d_stride_k = ctx->V_d;
    v.draft_ids = reinterpret_cast<const int32_t *>(d + L.draft);
    v.temperature = reinterpret_cast<const float *>(d + L.tau);
    v.uniforms = reinterpret_cast<const float *>(d + L.u);
    v.accepted = reinterpret_cast<int32_t *>(d + L.out);
    v.next_token = reinterpret_cast<int32_t *>(d + L.out) + B;
    v.row_status = reinterpret_cast<int32_t *>(d + L.status);
    v.workspace = d + L.ws; v.workspace_bytes = L.total - L.ws;
    const int rc = verify_impl(ctx, &v, cuda_stream, nullptr);
    if (rc != TLI_OK) return rc;
    if ((e = cudaMemcpyAsync(a->accepted, v.accepted, sizeof(int) * B, cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(a->next_token, v.next_token, sizeof(int) * B, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(e, "cudaMemcpyAsync to the host");
    if (a->row_status &&
        (e = cudaMemcpyAsync(a->row_status, v.row_status, sizeof(int) * B, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(e, "cudaMemcpyAsync to the host");
    return TLI_OK;
}

const char *tli_status_string(int code) {
    switch (code) {
        case TLI_OK: return "ok";
        case TLI_ERR_ARG: return "bad argument";
        case TLI_ERR_BAD_MAP: return "id map out of range or not injective";
        case TLI_ERR_CUDA: return "CUDA runtime error";
        case TLI_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case TLI_ERR_UNSUPPORTED: return "size beyond the library's limits";
        case TLI_ERR_STATIC_SCRATCH: return "batch needs more scratch than the built-in TLI_STATIC_SCRATCH_BYTES";
        default: return "unknown code";
    }
}

const char *tli_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"
