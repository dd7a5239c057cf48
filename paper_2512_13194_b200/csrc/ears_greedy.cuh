// The temperature -> 0 limit of the verification step (the deterministic regime named in
// Sec. 1): every softmax is one-hot at its row's largest logit, max P_t = 1, the tolerance
// beta (1 - max P_t) of Sec. 3.2 vanishes, and a greedily drafted token is accepted iff it is
// the top token of its target row.  The first mismatch ends the accepted prefix [Sec. 3.1]; the
// token emitted there (or after K acceptances) is the top token of that target row.  Only the
// target rows are read; no random numbers are drawn.
//
// A row is cut into pieces; CTAs stream pieces with 16-byte loads (several in flight per
// thread), keep (largest value, its smallest index) per thread, reduce per CTA and store one
// partial result per piece.  The CTA that delivers a sequence's last piece (an atomic ticket)
// combines the pieces per row and writes the outputs.  Nothing waits for anything.
#pragma once
#include <climits>

#include "ears_common.cuh"
#include "ears_math.cuh"
#include "ears_pipeline.cuh"

namespace ears {

#ifndef EARS_G_THREADS
#define EARS_G_THREADS 256
#endif
#ifndef EARS_G_CTAS
#define EARS_G_CTAS 3
#endif
#ifndef EARS_G_UNROLL
#define EARS_G_UNROLL 8
#endif
constexpr int kGThreads = EARS_G_THREADS;
constexpr int kGCtasPerSm = EARS_G_CTAS;
constexpr int kGUnroll = EARS_G_UNROLL;   // 16-byte loads in flight per thread

struct GParams {
    const void* t;        // target logits [B,K+1,V]
    const int32_t* x;     // draft tokens [B,K]
    int B, K, V;
    int P;                // pieces per row
    int piece_elems;      // entries per piece, a multiple of 256
    int vec;              // 1: rows are 16-byte aligned, vector loads
    long long units;      // B (K+1) P
    int4* partial;        // [units] (value bits, index, bad, -)
    int* ticket;          // [B] pieces of the sequence that are in
    int* heads;           // [2] status word
    int32_t* out_len;
    int32_t* out_tok;
    int* zero_ptr;        // counter block of the next call (see the host side)
    int zero_words;
};

struct Top { float v; int i; int bad; };

// larger value wins; among equal values the smaller index (the first of equal logits)
__device__ __forceinline__ void top_merge(Top& a, float v, int i, int bad) {
    if (v > a.v || (v == a.v && i < a.i)) { a.v = v; a.i = i; }
    a.bad |= bad;
}
__device__ __forceinline__ void top_take(Top& a, float v, int i) {
    if (v > a.v) { a.v = v; a.i = i; }   // entries arrive in increasing index order within a thread
    a.bad |= (v != v) ? 1 : 0;           // NaN
}

__device__ __forceinline__ uint4 load_stream16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

template <typename E> struct GVec;
template <> struct GVec<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void take(Top& a, uint4 w, int i0) {
        top_take(a, __uint_as_float(w.x), i0);
        top_take(a, __uint_as_float(w.y), i0 + 1);
        top_take(a, __uint_as_float(w.z), i0 + 2);
        top_take(a, __uint_as_float(w.w), i0 + 3);
    }
};
template <> struct GVec<uint16_t> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void take(Top& a, uint4 w, int i0) {
        top_take(a, __uint_as_float(w.x << 16), i0);     top_take(a, __uint_as_float(w.x & 0xffff0000u), i0 + 1);
        top_take(a, __uint_as_float(w.y << 16), i0 + 2); top_take(a, __uint_as_float(w.y & 0xffff0000u), i0 + 3);
        top_take(a, __uint_as_float(w.z << 16), i0 + 4); top_take(a, __uint_as_float(w.z & 0xffff0000u), i0 + 5);
        top_take(a, __uint_as_float(w.w << 16), i0 + 6); top_take(a, __uint_as_float(w.w & 0xffff0000u), i0 + 7);
    }
};
template <> struct GVec<f16_t> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void take(Top& a, uint4 w, int i0) {
        float x[8];
        Vec<f16_t>::unpack(w, x);
#pragma unroll
        for (int i = 0; i < 8; ++i) top_take(a, x[i], i0 + i);
    }
};

// One warp: combines the pieces of every target row of sequence b, compares the draft tokens
// with the rows' top tokens and writes accept length and tokens.
__device__ void greedy_finish(const GParams& p, int b, int lane, int* row_top /* shared, K+1 ints */) {
    const int K = p.K, P = p.P;
    bool bad = false;
    for (int k = lane; k <= K; k += 32) {
        Top a{-INFINITY, INT_MAX, 0};
        const int4* pp = p.partial + ((size_t)b * (K + 1) + k) * P;
        for (int j = 0; j < P; ++j) {
            const int4 q = __ldcg(pp + j);
            top_merge(a, __int_as_float(q.x), q.y, q.z);
        }
        // unusable row: a NaN, a +inf, or nothing finite (then no entry ever beat -inf)
        if (a.bad || a.v == INFINITY || a.i == INT_MAX) bad = true;
        row_top[k] = a.i;
    }
    __syncwarp();
    int first_miss = K;
    for (int k0 = 0; k0 < K; k0 += 32) {
        const int k = k0 + lane;
        bool miss = false;
        if (k < K) {
            const int tok = p.x[(size_t)b * K + k];
            if (tok < 0 || tok >= p.V) bad = true;
            miss = tok != row_top[k];
        }
        const unsigned m = __ballot_sync(0xffffffffu, miss);
        if (m != 0 && first_miss == K) first_miss = k0 + __ffs(m) - 1;
    }
    bad = __any_sync(0xffffffffu, bad);
    int32_t* ot = p.out_tok + (size_t)b * (K + 1);
    if (bad) {
        for (int j = lane; j <= K; j += 32) ot[j] = -1;
        if (lane == 0) {
            p.out_len[b] = -1;
            atomicOr(&p.heads[2], kDevInvalidInput);
            atomicAdd(&p.heads[kCountInvalid], 1);
        }
        return;
    }
    const int n = first_miss;
    for (int j = lane; j <= K; j += 32) ot[j] = j < n ? p.x[(size_t)b * K + j] : (j == n ? row_top[n] : -1);
    if (lane == 0) p.out_len[b] = n;
}

template <typename E>
__global__ void __launch_bounds__(kGThreads, kGCtasPerSm) ears_greedy_kernel(const GParams p) {
    constexpr int N = GVec<E>::N;
    // two copies, used alternately: one barrier per unit suffices, because a copy is rewritten only
    // after warp 0, which reads it, has arrived at the next unit's barrier
    __shared__ float s_v[2][kGThreads / 32];
    __shared__ int s_i[2][kGThreads / 32];
    __shared__ int s_bad[2][kGThreads / 32];
    __shared__ int s_top[kMaxK + 1];
    clear_next_counters(p);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = p.K, V = p.V, P = p.P;
    const E* base = reinterpret_cast<const E*>(p.t);
    int it = 0;
    for (long long u = blockIdx.x; u < p.units; u += gridDim.x, ++it) {
        const int h = it & 1;
        const long long row = u / P;
        const int piece = (int)(u % P);
        const int b = (int)(row / (K + 1));
        const int e0 = piece * p.piece_elems, e1 = min(V, e0 + p.piece_elems);
        const E* src = base + (size_t)row * V;
        Top a{-INFINITY, INT_MAX, 0};
        if (p.vec) {
            const int nvec = (e1 - e0) / N;   // V and piece_elems are multiples of N here
            const uint4* vs = reinterpret_cast<const uint4*>(src + e0);
            int v = tid;
            for (; v + (kGUnroll - 1) * kGThreads < nvec; v += kGUnroll * kGThreads) {
                uint4 w[kGUnroll];
#pragma unroll
                for (int j = 0; j < kGUnroll; ++j) w[j] = load_stream16(vs + v + j * kGThreads);
#pragma unroll
                for (int j = 0; j < kGUnroll; ++j) GVec<E>::take(a, w[j], e0 + (v + j * kGThreads) * N);
            }
            for (; v < nvec; v += kGThreads) GVec<E>::take(a, load_stream16(vs + v), e0 + v * N);
        } else {
            for (int i = e0 + tid; i < e1; i += kGThreads) top_take(a, load_logit(src + i), i);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, a.v, off);
            const int oi = __shfl_xor_sync(0xffffffffu, a.i, off);
            const int ob = __shfl_xor_sync(0xffffffffu, a.bad, off);
            top_merge(a, ov, oi, ob);
        }
        if (lane == 0) { s_v[h][warp] = a.v; s_i[h][warp] = a.i; s_bad[h][warp] = a.bad; }
        __syncthreads();
        if (warp == 0) {
            Top c{-INFINITY, INT_MAX, 0};
            if (lane < kGThreads / 32) c = Top{s_v[h][lane], s_i[h][lane], s_bad[h][lane]};
#pragma unroll
            for (int off = kGThreads / 64; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, c.v, off);
                const int oi = __shfl_xor_sync(0xffffffffu, c.i, off);
                const int ob = __shfl_xor_sync(0xffffffffu, c.bad, off);
                top_merge(c, ov, oi, ob);
            }
            int last = 0;
            if (lane == 0) {
                p.partial[u] = make_int4(__float_as_int(c.v), c.i, c.bad, 0);
                last = ticket_add(&p.ticket[b]) == (K + 1) * P - 1 ? 1 : 0;   // release the piece, acquire the others
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence();
                greedy_finish(p, b, lane, s_top);
            }
        }
    }
}

}  // namespace ears
