// Shapes, launch plan and workspace layout shared by the kernel and the host API.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace ears {

#ifndef EARS_CONSUMER_WARPS
#define EARS_CONSUMER_WARPS 8
#endif
#ifndef EARS_CTAS_PER_SM
#define EARS_CTAS_PER_SM 2
#endif
#ifndef EARS_STAGES
#define EARS_STAGES 6
#endif
constexpr int kConsumerWarps = EARS_CONSUMER_WARPS;  // warps that reduce the staged chunks
constexpr int kCtasPerSm = EARS_CTAS_PER_SM;
constexpr int kStages = EARS_STAGES;                 // 16 KB slots in a CTA's ring
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kLoaderWarp = kConsumerWarps;          // streams logits into shared memory
constexpr int kEpilogueWarp = kConsumerWarps + 1;    // counts finished pieces of rows
constexpr int kSequenceWarp = kConsumerWarps + 2;    // per-sequence decisions and the final pick
constexpr int kThreads = kConsumers + 96;
constexpr int kChunkBytes = 16384;                   // bytes staged per pipeline slot
constexpr int kSegElems = 256;                       // elements per final-token segment sum
constexpr int kMaxK = 64;                            // largest K (EARS_MAX_K of the C ABI)
constexpr double kEps = 1e-10;                       // division guard, Sec. 3.3 item 2
constexpr double kTinyMass = 1e-300;                 // below this a residual is treated as empty

// Device status bits (mirrors ears.h)
constexpr int kDevInvalidInput = 1;
constexpr int kDevTimeout = 2;

// Words of the `heads` block (16 ints at the start of every workspace) that every kernel shares:
// [2] the status word; [8..11] how the call's positions were decided, counted over what each
// sequence really decided (up to and including its first rejection): direct acceptances,
// pardons, rejections [Sec. 3.2 step 5], and [11] sequences marked invalid.
constexpr int kHeadsWords = 16;
constexpr int kCountDirect = 8, kCountPardon = 9, kCountReject = 10, kCountInvalid = 11;

// One warp: classes cls(k) in {0 reject, 1 direct, 2 pardon} of positions k < upto are added to the
// call's counters (cls_of: int(int k), evaluated by lane k % 32).
template <class F>
__device__ __forceinline__ void count_decisions(int* heads, int upto, int lane, F cls_of) {
    int nd = 0, np = 0, nr = 0;
    for (int k0 = 0; k0 < upto; k0 += 32) {
        const int k = k0 + lane;
        const int c = k < upto ? cls_of(k) : -1;
        nd += __popc(__ballot_sync(0xffffffffu, c == 1));
        np += __popc(__ballot_sync(0xffffffffu, c == 2));
        nr += __popc(__ballot_sync(0xffffffffu, c == 0));
    }
    if (lane == 0) {
        if (nd) atomicAdd(&heads[kCountDirect], nd);
        if (np) atomicAdd(&heads[kCountPardon], np);
        if (nr) atomicAdd(&heads[kCountReject], nr);
    }
}

// Sum of exp2(l c - mu) over one consumer warp's share of a chunk of the extra target row; mu is
// the fp32 product (running maximum) x c that the terms were taken relative to.
struct BonusSeg { double sum; float mu; float pad; };

struct Plan {
    int use_tma;   // 1: bulk asynchronous copies, 0: element-wise loader
    int parts1;    // pieces per row in the statistics pass
    int cpp1;      // chunks per piece
    int parts2;    // pieces per row in the final-token pass
    int job_elems; // elements of each row per piece of the final-token pass
    int nseg;      // segment sums per sequence
};

// Counter block at the start of the workspace, zeroed by one memset per call:
//   heads[8] (unit queue head, finalised sequences, status, published sequences,
//   sequence-work queue tail and head), wq[2B],
//   ticket1[B], ticket2[B], job_ctr[B], ticket_row[B*(2K+1)], ready[B].
struct Params {
    const void* t;        // target logits [B,K+1,V]
    const void* d;        // draft logits  [B,K,V]
    const int32_t* x;     // draft tokens  [B,K]
    int B, K, V;
    float c;              // log2(e) / temperature
    double T;             // temperature
    double beta;
    const float* seq_T;   // [B] per-sequence temperature, or NULL (then T for all)
    const float* seq_beta;  // [B] per-sequence beta, or NULL
    unsigned long long seed, offset;
    long long b_first;
    int32_t* out_len;     // [B]
    int32_t* out_tok;     // [B,K+1]
    double* pt_tok;       // [B,K]
    double* pd_tok;       // [B,K]
    double* max_pt;       // [B,K]
    uint8_t* cls;         // [B,K]
    double* resid;        // [B]
    int* ticket1;         // [B] rows of the sequence whose pieces are all in
    int* ticket_row;      // [B*(2K+1)] pieces of the row that are in
    int* ticket2;         // [B] final-token pieces of the sequence that are in
    unsigned long long* ready;  // [B] published sequences: (b + 1) << 32 | n, 0 = not yet
    int* job_ctr;         // [B] final-token pieces handed out, per published slot
    int* heads;           // [0] unit queue, [1] finalised sequences, [2] status, [3] published sequences,
                          // [4] / [5] tail / head of the sequence-work queue
    unsigned long long* wq;  // [2B] sequence work: bit 63 valid, bits 32..62 sequence, low word n or ~0 (decide)
    float2* partial;      // [B*(2K+1)*parts1] (m, s) per row piece
    float2* rowstat;      // [B*(2K+1)] (m, Z) per row
    // Per sequence one region of seg_stride bytes, used first for the extra row's BonusSeg
    // entries [chunks*8] and, if a position is rejected, afterwards for the second pass's
    // segment sums (double [nseg]); a sequence never needs both at once.
    unsigned char* seg_base;
    size_t seg_stride;
    int stop_first;       // 1: what lies after a sequence's first rejection is neither validated nor reported
    int unc_entropy;      // 1: the tolerance is scaled by H(P_t) / ln V instead of 1 - max P_t [Sec. 5 item 1]
    double* entropy;      // [B,K] H(P_t) of every target row, or NULL; the entropy kernels (ENT) fill it
    float* partial_w;     // [B*(2K+1)*parts1] sum e t per row piece (ENT kernels)
    float* roww;          // [B*(2K+1)] sum e t per row (ENT kernels)
    int* zero_ptr;        // counter block of the next call, cleared by this kernel (zero_words ints; may be 0)
    int zero_words;
    Plan plan;
};

// All threads of the grid clear the other copy of the counter block (see the host side).
template <class P> __device__ __forceinline__ void clear_next_counters(const P& p) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < p.zero_words; i += gridDim.x * blockDim.x) p.zero_ptr[i] = 0;
}

// Temperature and base tolerance of (local) sequence b: the per-sequence arrays where given,
// else the call's scalars.  c = log2(e) / T is formed the way the host forms it for the scalar.
template <class P> __device__ __forceinline__ double seq_temperature(const P& p, int b) {
    return p.seq_T ? (double)__ldg(p.seq_T + b) : p.T;
}
template <class P> __device__ __forceinline__ double seq_beta(const P& p, int b) {
    return p.seq_beta ? (double)__ldg(p.seq_beta + b) : p.beta;
}
// (kept out of line: the fp64 division would otherwise sit in every role's hot loop, and the
// streaming kernel is sensitive to the size of those loops)
__device__ __noinline__ float seq_c_from_array(const float* seq_T, int b) {
    return (float)(1.4426950408889634 / (double)__ldg(seq_T + b));
}
template <class P> __device__ __forceinline__ float seq_c(const P& p, int b) {
    return p.seq_T ? seq_c_from_array(p.seq_T, b) : p.c;
}
// What the host refuses in the scalar form makes a sequence invalid in the per-sequence form.
__device__ __forceinline__ bool seq_params_ok(double T, double beta) {
    return T > 0.0 && T < 1e300 && beta >= 0.0 && beta < 1e300;   // NaN fails every comparison
}

__host__ __device__ inline double* seg_sums(const Params& p, int b) { return reinterpret_cast<double*>(p.seg_base + (size_t)b * p.seg_stride); }
__host__ __device__ inline BonusSeg* bonus_segs(const Params& p, int b) { return reinterpret_cast<BonusSeg*>(p.seg_base + (size_t)b * p.seg_stride); }

// Row order inside a sequence: target k, draft k for k = 0..K-1, then the bonus
// target row K.  ridx in [0, 2K].
__host__ __device__ inline long long target_row(int b, int k, int K) { return (long long)b * (K + 1) + k; }
__host__ __device__ inline long long draft_row(int b, int k, int K) { return (long long)b * K + k; }

}  // namespace ears
