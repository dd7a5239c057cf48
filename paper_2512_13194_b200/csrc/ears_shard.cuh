// Verification with the vocabulary split across devices (tensor-parallel logits): every device
// holds the columns [v_first, v_first + Vs) of every row.  The step of Sec. 3.2 needs, per row,
// only the maximum, the normaliser and the logit of the draft token; the final draw of Sec. 3.1
// needs, per sequence, the mass each device holds of the one row (pair) that is drawn from.  So the
// step runs in three local phases with two small exchanges between them:
//   1. statistics of the local columns of every row: (m, s = sum exp2((l - m) c), logit of the
//      draft token if it lies here)                        -> exchange: 16 bytes per row
//   2. every device combines all devices' statistics in the same order (bitwise identical
//      decisions everywhere), finds the first rejection, and sums the local mass of the row to
//      draw from: max(0, P_t - P_d) after a rejection, P_t after K acceptances, in 256-entry
//      segments                                            -> exchange: 8 bytes per sequence
//   3. the device whose columns contain the point u * S of the cumulative mass (devices in
//      vocabulary order) picks the token; the others write -1; a MAX over devices finishes.
// Logits never leave the device that holds them.
#pragma once
#include "ears_common.cuh"
#include "ears_direct.cuh"
#include "ears_kernel.cuh"
#include "ears_math.cuh"
#include "ears_philox.cuh"

namespace ears {

constexpr int kSThreads = kDThreads;     // stream_piece strides over this many threads
constexpr int kSCtasPerSm = 3;
constexpr int kSSegsPerCta = 64;         // 256-entry segments per CTA in the mass pass
constexpr int kSSeqPerCta = 4;           // one warp per sequence in the decision and pick kernels

struct SParams {
    const void* t;         // target columns [B,K+1,Vs]
    const void* d;         // draft columns  [B,K,Vs]
    const int32_t* x;      // draft tokens [B,K], ids of the whole vocabulary
    int B, K, Vs, V;       // V: whole vocabulary
    int v_first;           // id of local column 0
    int n_shards;
    int P, piece_elems, vec;
    float c;               // log2(e) / temperature
    double T, beta;
    unsigned long long seed, offset;
    long long b_first;
    float4* stats;             // phase 1 result [B (2K+1)]: (m, s, token logit, 1 if the token lies here)
    const float4* all_stats;   // [n_shards][B (2K+1)]
    const double* all_mass;    // [n_shards][B]
    double* mass;              // phase 2 result [B]
    int32_t* out_len;
    int32_t* out_tok;
    int* ticket_row;       // [B (2K+1)]
    int* ticket_seq;       // [B]
    float2* partial;       // [B (2K+1) P]
    float4* rowstat;       // [B (2K+1)] combined (M, Z, token logit, number of devices that claimed the token)
    int* sel;              // [B] accepted length, -1 for an invalid sequence
    double* seg;           // [B][nseg] local segment sums of the row to draw from
    int nseg;
};

// rows of a sequence: r in [0, K] target row r, r in (K, 2K] draft row r - K - 1
template <typename E>
__device__ __forceinline__ const E* shard_row(const SParams& p, int b, int r) {
    return r <= p.K ? reinterpret_cast<const E*>(p.t) + ((size_t)b * (p.K + 1) + r) * p.Vs
                    : reinterpret_cast<const E*>(p.d) + ((size_t)b * p.K + (r - p.K - 1)) * p.Vs;
}

// ---- phase 1 ----------------------------------------------------------------------
// The draft token of row r of sequence b if its column is local, else -1 (the extra target row
// has none).
__device__ __forceinline__ int shard_local_token(const SParams& p, long long row) {
    const int K = p.K, R = 2 * K + 1;
    const int b = (int)(row / R), r = (int)(row % R);
    if (r == K) return -1;
    const int tok = __ldg(p.x + (size_t)b * K + (r < K ? r : r - K - 1));
    return (tok >= p.v_first && tok - p.v_first < p.Vs) ? tok - p.v_first : -1;
}

template <typename E>
__global__ void __launch_bounds__(kSThreads, kSCtasPerSm) ears_shard_stats_kernel(const SParams p) {
    __shared__ float2 s_ms[2][kSThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, R = 2 * K + 1, P = p.P;
    const long long units = (long long)p.B * R * P;
    // thread 0 finishes rows; it fetches the token one unit ahead and the token's logit at the
    // start of the unit, so that neither load is waited for at the end
    int tok_next = (tid == 0 && blockIdx.x < units) ? shard_local_token(p, blockIdx.x / P) : -1;
    int it = 0;
    for (long long u = blockIdx.x; u < units; u += gridDim.x, ++it) {
        const long long row = u / P;
        const int piece = (int)(u % P);
        const int b = (int)(row / R), r = (int)(row % R);
        const E* src = shard_row<E>(p, b, r);
        const int e0 = piece * p.piece_elems, e1 = min(p.Vs, e0 + p.piece_elems);
        const int tok = tok_next;
        float l = 0.f;
        if (tid == 0) {
            if (tok >= 0) l = load_logit(src + tok);
            tok_next = u + gridDim.x < units ? shard_local_token(p, (u + gridDim.x) / P) : -1;
        }
        float2 ms = stream_piece<E>(src, e0, e1, p.vec != 0, p.c, tid);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, ms.x, off);
            const float os = __shfl_xor_sync(0xffffffffu, ms.y, off);
            merge_ms(ms.x, ms.y, om, os, p.c);
        }
        if (lane == 0) s_ms[it & 1][warp] = ms;
        // one barrier per unit: the other half of s_ms is rewritten only after thread 0, which
        // reads this half below, has reached the next unit's barrier
        __syncthreads();
        if (tid == 0) {
            float m = -INFINITY, s = 0.f;
            for (int i = 0; i < kSThreads / 32; ++i) merge_ms(m, s, s_ms[it & 1][i].x, s_ms[it & 1][i].y, p.c);
            bool last = true;
            if (P > 1) {
                p.partial[u] = make_float2(m, s);
                last = ticket_add(&p.ticket_row[row]) == P - 1;   // releases this piece, acquires the others
                if (last) {
                    m = -INFINITY; s = 0.f;
                    for (int i = 0; i < P; ++i) {
                        const float2 q = __ldcg(p.partial + row * P + i);
                        merge_ms(m, s, q.x, q.y, p.c);
                    }
                }
            }
            if (last) p.stats[row] = make_float4(m, s, tok >= 0 ? l : 0.f, tok >= 0 ? 1.f : 0.f);
        }
    }
}

// Short rows: one warp per row, no block-wide step at all (eight rows in flight per CTA).
template <typename E>
__global__ void __launch_bounds__(kSThreads, kSCtasPerSm) ears_shard_stats_rows_kernel(const SParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int K = p.K, R = 2 * K + 1;
    const long long rows = (long long)p.B * R;
    for (long long row = (long long)blockIdx.x * (kSThreads / 32) + warp; row < rows; row += (long long)gridDim.x * (kSThreads / 32)) {
        const int b = (int)(row / R), r = (int)(row % R);
        const E* src = shard_row<E>(p, b, r);
        const int tok = lane == 0 ? shard_local_token(p, row) : -1;
        const float l = tok >= 0 ? load_logit(src + tok) : 0.f;   // in flight during the sweep
        float2 ms = stream_piece<E, 32>(src, 0, p.Vs, p.vec != 0, p.c, lane);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, ms.x, off);
            const float os = __shfl_xor_sync(0xffffffffu, ms.y, off);
            merge_ms(ms.x, ms.y, om, os, p.c);
        }
        if (lane == 0) p.stats[row] = make_float4(ms.x, ms.y, tok >= 0 ? l : 0.f, tok >= 0 ? 1.f : 0.f);
    }
}

// ---- phase 2a: decisions, identical on every device ---------------------------------
__global__ void __launch_bounds__(kSSeqPerCta * 32) ears_shard_decide_kernel(const SParams p) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kSSeqPerCta + (threadIdx.x >> 5);
    if (b >= p.B) return;
    const int K = p.K, R = 2 * K + 1;
    const size_t rows = (size_t)p.B * R;
    bool bad = false;
    for (int r = lane; r < R; r += 32) {
        float m = -INFINITY, s = 0.f, l = 0.f;
        int owners = 0;
        for (int sh = 0; sh < p.n_shards; ++sh) {
            const float4 q = __ldg(p.all_stats + sh * rows + (size_t)b * R + r);
            merge_ms(m, s, q.x, q.y, p.c);
            if (q.w != 0.f) { l = q.z; ++owners; }
        }
        if (!rowstat_ok(m, s)) bad = true;
        p.rowstat[(size_t)b * R + r] = make_float4(m, s, l, (float)owners);
    }
    __syncwarp();
    int first_reject = K;
    for (int k0 = 0; k0 < K; k0 += 32) {
        const int k = k0 + lane;
        bool reject = false;
        if (k < K) {
            const int tok = p.x[(size_t)b * K + k];
            const float4 qt = p.rowstat[(size_t)b * R + k];
            const float4 qd = p.rowstat[(size_t)b * R + K + 1 + k];
            if (tok < 0 || tok >= p.V || qt.w != 1.f || qd.w != 1.f) {
                bad = true;   // no device, or more than one, holds the token's column
            } else {
                const double U = uniform_accept(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)k);
                const Decision dc = decide_position((double)qt.z, (double)qd.z, make_float2(qt.x, qt.y),
                                                    make_float2(qd.x, qd.y), p.T, p.beta, U);
                reject = !dc.accept;
            }
        }
        const unsigned rej = __ballot_sync(0xffffffffu, reject);
        if (rej != 0 && first_reject == K) first_reject = k0 + __ffs(rej) - 1;
    }
    bad = __any_sync(0xffffffffu, bad);
    int32_t* ot = p.out_tok + (size_t)b * (K + 1);
    if (bad) {
        for (int j = lane; j <= K; j += 32) ot[j] = -1;
        if (lane == 0) { p.out_len[b] = -1; p.sel[b] = -1; p.mass[b] = 0.0; }
        return;
    }
    for (int j = lane; j <= K; j += 32) ot[j] = j < first_reject ? p.x[(size_t)b * K + j] : -1;
    if (lane == 0) { p.out_len[b] = first_reject; p.sel[b] = first_reject; }
}

// Masses of the eight entries base + 8 lane .. + 7 of a segment, summed in index order (fp64).
// Entries beyond the local columns count as -inf logits (no mass).
template <typename E, bool RESID>
__device__ __forceinline__ double lane_mass8(const E* trow, const E* drow, int base, int Vs, bool vec,
                                             const RowNorm& rn, float c, int lane) {
    constexpr int N = Words<E>::N;
    double sum = 0.0;
#pragma unroll
    for (int j = 0; j < 8 / N; ++j) {
        const int e = base + lane * 8 + j * N;
        const int left = Vs - e;
        uint4 wt, wd = Words<E>::minus_inf();
        if (vec && left >= N) {
            wt = ld_stream16(trow + e);
            if (RESID) wd = ld_stream16(drow + e);
        } else {
            wt = Words<E>::gather(trow + e, left);
            if (RESID) wd = Words<E>::gather(drow + e, left);
        }
        float xt[N], xd[N];
        Words<E>::unpack(wt, xt);
        Words<E>::unpack(wd, xd);
#pragma unroll
        for (int i = 0; i < N; ++i) sum += (double)entry_mass<RESID>(xt[i], xd[i], rn, c);
    }
    return sum;
}

__device__ __forceinline__ RowNorm shard_rownorm(const SParams& p, int b, int n) {
    const int K = p.K, R = 2 * K + 1;
    const float4 qt = __ldcg(p.rowstat + (size_t)b * R + n);
    const float4 qd = n < K ? __ldcg(p.rowstat + (size_t)b * R + K + 1 + n) : qt;
    return make_rownorm(make_float2(qt.x, qt.y), make_float2(qd.x, qd.y));
}

// ---- phase 2b: local mass of the row each sequence draws from -------------------------
template <typename E>
__global__ void __launch_bounds__(kSThreads) ears_shard_mass_kernel(const SParams p, int ctas_per_seq) {
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / ctas_per_seq, j = blockIdx.x % ctas_per_seq;
    const int n = __ldcg(p.sel + b);
    if (n < 0) return;
    const int K = p.K;
    const bool resid = n < K;
    const E* trow = shard_row<E>(p, b, n);
    const E* drow = resid ? shard_row<E>(p, b, K + 1 + n) : trow;
    const RowNorm rn = shard_rownorm(p, b, n);
    const int g1 = min(p.nseg, (j + 1) * kSSegsPerCta);
    for (int g = j * kSSegsPerCta + warp; g < g1; g += kSThreads / 32) {
        const double mine = resid ? lane_mass8<E, true>(trow, drow, g * kSegElems, p.Vs, p.vec != 0, rn, p.c, lane)
                                  : lane_mass8<E, false>(trow, drow, g * kSegElems, p.Vs, p.vec != 0, rn, p.c, lane);
        const double incl = warp_inclusive_scan(mine, lane);
        if (lane == 31) {
            p.seg[(size_t)b * p.nseg + g] = incl;
            __threadfence();
        }
    }
    __syncthreads();
    if (tid == 0) s_last = ticket_add(&p.ticket_seq[b]) == ctas_per_seq - 1 ? 1 : 0;
    __syncthreads();
    if (!s_last || warp != 0) return;
    __threadfence();
    // the sequence's last CTA: segment sums in index order (lanes own contiguous blocks)
    const int per = (p.nseg + 31) / 32;
    const int a0 = min(p.nseg, lane * per), a1 = min(p.nseg, a0 + per);
    double loc = 0.0;
    for (int g = a0; g < a1; ++g) loc += __ldcg(p.seg + (size_t)b * p.nseg + g);
    const double incl = warp_inclusive_scan(loc, lane);
    if (lane == 31) p.mass[b] = incl;
}

// Absolute point `tin` of the cumulative P_t mass of local columns [0, Vs) of one row: the first
// entry whose running sum exceeds it (the last entry with mass if rounding hides the crossing).
template <typename E>
__device__ int warp_walk_pt(const E* row, int Vs, const RowNorm& rn, float c, double tin, int lane) {
    const int per = (Vs + 31) / 32;
    const int v0 = min(Vs, lane * per), v1 = min(Vs, v0 + per);
    double loc = 0.0;
    for (int v = v0; v < v1; ++v) loc += (double)entry_mass<false>(load_logit(row + v), 0.f, rn, c);
    const double inc = warp_inclusive_scan(loc, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, tin < inc && loc > 0.0);
    const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
    if (!pos) return -1;
    const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
    int tok = -1;
    if (lane == L) {
        double cum = inc - loc;
        int lastpos = -1;
        for (int v = v0; v < v1; ++v) {
            const double r = (double)entry_mass<false>(load_logit(row + v), 0.f, rn, c);
            if (r > 0.0) lastpos = v;
            cum += r;
            if (tin < cum && r > 0.0) { tok = v; break; }
        }
        if (tok < 0) tok = lastpos;
    }
    return __shfl_sync(0xffffffffu, tok, L);
}

// Which device's columns contain the point u * S (devices in vocabulary order)?  value(sh) is
// device sh's mass.  -> device, and the point relative to the start of its columns.
template <typename F>
__device__ __forceinline__ int owner_of(F value, int n_shards, double u, double* tin_out, double* S_out) {
    double S = 0.0;
    for (int sh = 0; sh < n_shards; ++sh) S += value(sh);
    const double target = u * S;
    double cum = 0.0, before = 0.0, before_last = 0.0;
    int owner = -1, lastpos = -1;
    for (int sh = 0; sh < n_shards; ++sh) {
        const double v = value(sh);
        if (v > 0.0) { lastpos = sh; before_last = cum; }
        if (owner < 0 && v > 0.0 && target < cum + v) { owner = sh; before = cum; }
        cum += v;
    }
    if (owner < 0) { owner = lastpos; before = before_last; }
    *tin_out = target - before;
    *S_out = S;
    return owner;
}

// ---- phase 3: the final token ----------------------------------------------------------
template <typename E>
__global__ void __launch_bounds__(kSSeqPerCta * 32) ears_shard_pick_kernel(const SParams p, int shard) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kSSeqPerCta + (threadIdx.x >> 5);
    if (b >= p.B) return;
    const int K = p.K, R = 2 * K + 1;
    const int n = __ldcg(p.sel + b);
    if (n < 0) return;   // invalid: every slot already holds -1
    int32_t* slot = p.out_tok + (size_t)b * (K + 1) + n;
    const bool resid = n < K;
    const E* trow = shard_row<E>(p, b, n);
    const E* drow = resid ? shard_row<E>(p, b, K + 1 + n) : trow;
    const RowNorm rn = shard_rownorm(p, b, n);
    const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)K);
    double tin, S;
    int owner = owner_of([&](int sh) { return __ldg(p.all_mass + (size_t)sh * p.B + b); }, p.n_shards, u, &tin, &S);
    if (!(S >= kTinyMass)) {
        // a residual without mass cannot follow a rejection in exact arithmetic; draw from P_t,
        // whose mass per device is known from the statistics
        const size_t rows = (size_t)p.B * R;
        const float M = rn.mt;
        owner = owner_of([&](int sh) {
            const float4 q = __ldg(p.all_stats + sh * rows + (size_t)b * R + n);
            return (double)rebase_sum(q.x, q.y, M, p.c);
        }, p.n_shards, u, &tin, &S);
        int tok = -1;
        if (owner == shard) tok = warp_walk_pt<E>(trow, p.Vs, rn, p.c, tin, lane);
        if (lane == 0) *slot = tok >= 0 ? p.v_first + tok : -1;
        return;
    }
    if (owner != shard) {
        if (lane == 0) *slot = -1;
        return;
    }
    // first level: the segment (lanes own contiguous blocks of the stored segment sums)
    const double* seg = p.seg + (size_t)b * p.nseg;
    const int per = (p.nseg + 31) / 32;
    const int a0 = min(p.nseg, lane * per), a1 = min(p.nseg, a0 + per);
    double loc = 0.0;
    for (int g = a0; g < a1; ++g) loc += __ldcg(seg + g);
    const double incl = warp_inclusive_scan(loc, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, tin < incl && loc > 0.0);
    const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
    if (!pos) {   // the mass this device reported has no segment behind it: cannot happen
        if (lane == 0) *slot = -1;
        return;
    }
    const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
    int g_found = -1;
    double before = 0.0;
    if (lane == L) {
        double cum = incl - loc, before_last = 0.0;
        int lastg = -1;
        for (int g = a0; g < a1; ++g) {
            const double v = __ldcg(seg + g);
            if (v > 0.0) { lastg = g; before_last = cum; }
            if (v > 0.0 && tin < cum + v) { g_found = g; before = cum; break; }
            cum += v;
        }
        if (g_found < 0) { g_found = lastg; before = before_last; }
    }
    g_found = __shfl_sync(0xffffffffu, g_found, L);
    before = __shfl_sync(0xffffffffu, before, L);
    const int tok = pick_in_range<E>(trow, drow, resid, rn, p.c, g_found * kSegElems, kSegElems, tin - before, p.Vs, lane);
    if (lane == 0) *slot = tok >= 0 ? p.v_first + tok : -1;
}

}  // namespace ears
