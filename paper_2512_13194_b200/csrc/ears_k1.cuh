// Kernel 1: row statistics, accept decisions and the first-rejection scan.
//
// Every logits row is read once.  A row is cut into pieces ("units"); persistent
// CTAs pull units from an atomic queue.  Inside a CTA one loader warp streams the
// unit through a ring of shared-memory slots (bulk asynchronous copies completing
// on mbarriers, or an element-wise copy when the data is not 16-byte aligned) and
// eight consumer warps keep a running (max, sum of exp2) per thread.  The CTA that
// delivers the last piece of a sequence merges the pieces, forms P_t(x), P_d(x),
// max P_t = 1/Z_t, draws U_k, decides (Sec. 3.2) and scans for the first
// rejection (Sec. 3.1).  No CTA ever waits for another CTA.
#pragma once
#include "ears_common.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"

namespace ears {

struct StageMeta {
    int unit;    // -1: end of work
    int nelem;   // valid elements in the slot
    int flags;   // bit 0: first chunk of the unit, bit 1: last chunk of the unit
    int elem0;   // index of the slot's first element within its row
};

template <int STAGES, int ROWS_PER_SLOT>
struct PipeSmem {
    alignas(128) unsigned char buf[STAGES][ROWS_PER_SLOT][kChunkBytes];
    alignas(8) uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t red[STAGES];
    StageMeta meta[STAGES];
    int meta_aux[STAGES];
    float2 scratch[STAGES][kConsumerWarps];
    int abort_flag;
};

template <int STAGES, int ROWS_PER_SLOT>
__device__ __forceinline__ void pipe_init(PipeSmem<STAGES, ROWS_PER_SLOT>& sm, bool use_tma) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm.full[s], use_tma ? 1u : 32u);
            mbar_init(&sm.empty[s], kConsumerWarps);
            mbar_init(&sm.red[s], kConsumerWarps);
        }
        sm.abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
}

// Loader side: waits until slot `q % STAGES` is free.  Whole warp; uniform result.
template <int STAGES, int ROWS_PER_SLOT>
__device__ __forceinline__ bool loader_acquire(PipeSmem<STAGES, ROWS_PER_SLOT>& sm, uint32_t q, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(&sm.empty[q % STAGES], ((q / STAGES) & 1u) ^ 1u, &sm.abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Element-wise copy of n elements into a slot by the loader warp (unaligned data).
template <typename E>
__device__ __forceinline__ void lane_copy(void* dst, const E* src, int n, int lane) {
    E* o = reinterpret_cast<E*>(dst);
    for (int i = lane; i < n; i += 32) o[i] = __ldg(src + i);
}

// After an abort: give copies that may still be in flight a bounded time to land
// before the CTA's shared memory is released.
template <int STAGES, int ROWS_PER_SLOT>
__device__ __forceinline__ void loader_drain(PipeSmem<STAGES, ROWS_PER_SLOT>& sm, uint32_t issued) {
    uint32_t first = issued > STAGES ? issued - STAGES : 0;
    for (uint32_t q = first; q < issued; ++q) {
        unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(&sm.full[q % STAGES], (q / STAGES) & 1u)) {
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
    }
}

// ---- consumer arithmetic ---------------------------------------------------
template <typename E> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const unsigned char* buf, int vec_index, float (&x)[4]) {
        float4 v = reinterpret_cast<const float4*>(buf)[vec_index];
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};
template <> struct Vec<uint16_t> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const unsigned char* buf, int vec_index, float (&x)[8]) {
        uint4 v = reinterpret_cast<const uint4*>(buf)[vec_index];
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

__device__ __forceinline__ float load_logit(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_logit(const uint16_t* p) { return bf16_bits_to_float(__ldg(p)); }

// Running (m, s) of one thread over its share of a staged chunk:
// s = sum exp2((l - m) * c), m = running maximum; s is rescaled when m grows.
template <typename E>
__device__ __forceinline__ void chunk_stats(const unsigned char* buf, int nelem, int tid, float c,
                                            float& m_run, float (&s)[4]) {
    constexpr int N = Vec<E>::N;
    constexpr int VECS = kChunkBytes / 16 / kConsumers;  // 16-byte vectors per thread per chunk
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    float x[VECS][N];
#pragma unroll
    for (int j = 0; j < VECS; ++j) Vec<E>::load(buf, j * kConsumers + tid, x[j]);
    if (nelem < CHUNK_ELEMS) {  // ragged last chunk of a row: mask what lies beyond it
#pragma unroll
        for (int j = 0; j < VECS; ++j)
#pragma unroll
            for (int i = 0; i < N; ++i)
                if ((j * kConsumers + tid) * N + i >= nelem) x[j][i] = -INFINITY;
    }
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < VECS; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) cm = fmaxf(cm, x[j][i]);
    if (cm > m_run) {
        float sc = ex2_approx((m_run - cm) * c);  // m_run = -inf gives 0
        s[0] *= sc; s[1] *= sc; s[2] *= sc; s[3] *= sc;
        m_run = cm;
    }
    const float mu = (m_run == -INFINITY) ? 0.0f : m_run;
#pragma unroll
    for (int j = 0; j < VECS; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) s[(j * N + i) & 3] += ex2_approx(__fmul_rn(__fsub_rn(x[j][i], mu), c));
}

// ---- per-sequence epilogue (one warp) ----------------------------------------
// Merges the pieces of all 2K+1 rows, writes (m, Z) per row, decides every position
// (Sec. 3.2 steps 1-5 with the guards of Sec. 3.3 item 2) and writes the accepted
// prefix (Sec. 3.1).  The slot of the final token is filled by kernel 2.
template <typename E>
__device__ void finalize_sequence(const Params& p, int b, int lane) {
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1;
    const E* t = reinterpret_cast<const E*>(p.t);
    const E* d = reinterpret_cast<const E*>(p.d);
    bool bad = false;
    for (int r = lane; r < R; r += 32) {
        float m = -INFINITY, s = 0.0f;
        const float2* pp = p.partial + ((size_t)b * R + r) * P;
        for (int i = 0; i < P; ++i) {
            float2 v = __ldcg(pp + i);
            merge_ms(m, s, v.x, v.y, p.c);
        }
        if (!(m > -INFINITY && m < INFINITY && s > 0.0f && s < INFINITY)) bad = true;  // NaN fails too
        p.rowstat[(size_t)b * R + r] = make_float2(m, s);
    }
    __syncwarp();
    int first_reject = K;
    for (int k0 = 0; k0 < K; k0 += 32) {
        const int k = k0 + lane;
        bool reject = false;
        if (k < K) {
            const int tok = p.x[(size_t)b * K + k];
            if (tok < 0 || tok >= V) {
                bad = true;
            } else {
                const float2 st = __ldcg(&p.rowstat[(size_t)b * R + 2 * k]);
                const float2 sd = __ldcg(&p.rowstat[(size_t)b * R + 2 * k + 1]);
                const double lt = (double)load_logit(t + (size_t)target_row(b, k, K) * V + tok);
                const double ld = (double)load_logit(d + (size_t)draft_row(b, k, K) * V + tok);
                const double pt = exp((lt - (double)st.x) / p.T) / (double)st.y;
                const double pd = exp((ld - (double)sd.x) / p.T) / (double)sd.y;
                const double maxp = 1.0 / (double)st.y;                 // the largest term of Z is exp(0)
                const double ratio = pt / fmax(pd, kEps);               // R_k with the division guard
                const double tol = p.beta * (1.0 - maxp);               // Tolerance_k
                const double U = uniform_accept(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)k);
                const double thr = fmax(U - tol, 0.0);                  // clamped threshold
                const bool accept = ratio >= thr;
                reject = !accept;
                const size_t i = (size_t)b * K + k;
                p.pt_tok[i] = pt;
                p.pd_tok[i] = pd;
                p.max_pt[i] = maxp;
                p.cls[i] = ratio >= U ? 1 : (accept ? 2 : 0);
            }
        }
        const unsigned rej = __ballot_sync(0xffffffffu, reject);
        if (rej != 0 && first_reject == K) first_reject = k0 + __ffs(rej) - 1;
    }
    bad = __any_sync(0xffffffffu, bad);
    int32_t* ot = p.out_tok + (size_t)b * (K + 1);
    if (bad) {
        for (int j = lane; j <= K; j += 32) ot[j] = -1;
        if (lane == 0) {
            p.out_len[b] = -1;
            atomicOr(&p.heads[2], kDevInvalidInput);
        }
    } else {
        for (int j = lane; j <= K; j += 32) ot[j] = j < first_reject ? p.x[(size_t)b * K + j] : -1;
        if (lane == 0) p.out_len[b] = first_reject;
    }
}

// ---- the kernel -------------------------------------------------------------
template <typename E, int STAGES>
__global__ void __launch_bounds__(kThreads, 2) k1_rowstats_decide(const Params p) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = PipeSmem<STAGES, 1>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1, cpp = p.plan.cpp1;
    const bool use_tma = p.plan.use_tma != 0;
    const int chunks_per_row = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    const long long total_units = (long long)p.B * R * P;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    pipe_init(sm, use_tma);

    if (warp == kConsumerWarps) {
        // ------------------------------ loader warp
        uint32_t q = 0;
        bool ok = true;
        while (ok) {
            long long u = 0;
            if (lane == 0) u = atomicAdd(&p.heads[0], 1);
            u = __shfl_sync(0xffffffffu, u, 0);
            if (u >= total_units || sm.abort_flag) break;
            const int b = (int)(u / (R * P));
            const int rem = (int)(u % (R * P));
            const int ridx = rem / P, part = rem % P;
            const E* row = (ridx == 2 * K)
                               ? reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, K, K) * V
                               : ((ridx & 1) ? reinterpret_cast<const E*>(p.d) + (size_t)draft_row(b, ridx >> 1, K) * V
                                             : reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, ridx >> 1, K) * V);
            const int ch0 = part * cpp;
            const int ch1 = min(chunks_per_row, ch0 + cpp);
            for (int ch = ch0; ch < ch1; ++ch, ++q) {
                ok = loader_acquire(sm, q, lane);
                if (!ok) break;
                const int stage = q % STAGES;
                const int e0 = ch * CHUNK_ELEMS;
                const int n = min(CHUNK_ELEMS, V - e0);
                if (lane == 0) sm.meta[stage] = StageMeta{(int)u, n, (ch == ch0 ? 1 : 0) | (ch == ch1 - 1 ? 2 : 0), e0};
                if (use_tma) {
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&sm.full[stage], (uint32_t)n * (uint32_t)sizeof(E));
                        bulk_load(sm.buf[stage][0], row + e0, (uint32_t)n * (uint32_t)sizeof(E), &sm.full[stage]);
                    }
                } else {
                    lane_copy<E>(sm.buf[stage][0], row + e0, n, lane);
                    __syncwarp();
                    mbar_arrive(&sm.full[stage]);
                }
            }
        }
        if (ok && loader_acquire(sm, q, lane)) {  // end-of-work marker
            const int stage = q % STAGES;
            if (lane == 0) sm.meta[stage] = StageMeta{-1, 0, 0, 0};
            __syncwarp();
            if (use_tma) { if (lane == 0) mbar_arrive(&sm.full[stage]); }
            else mbar_arrive(&sm.full[stage]);
        } else if (use_tma && lane == 0) {
            loader_drain(sm, q);
        }
    } else {
        // ------------------------------ consumer warps
        const int tid = threadIdx.x;
        float m_run = -INFINITY;
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t red_phase = 0;
        for (uint32_t q = 0;; ++q) {
            const int stage = q % STAGES;
            if (!mbar_wait(&sm.full[stage], (q / STAGES) & 1u, &sm.abort_flag)) break;
            const StageMeta mt = sm.meta[stage];
            if (mt.unit < 0) break;
            if (mt.flags & 1) { m_run = -INFINITY; s[0] = s[1] = s[2] = s[3] = 0.f; }
            chunk_stats<E>(sm.buf[stage][0], mt.nelem, tid, p.c, m_run, s);
            if (!(mt.flags & 2)) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[stage]);
                continue;
            }
            // last chunk of the unit: reduce the CTA's (m, s)
            float m = m_run, sum = (s[0] + s[1]) + (s[2] + s[3]);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                float m2 = __shfl_xor_sync(0xffffffffu, m, off);
                float s2 = __shfl_xor_sync(0xffffffffu, sum, off);
                merge_ms(m, sum, m2, s2, p.c);
            }
            if (lane == 0) {
                sm.scratch[stage][warp] = make_float2(m, sum);
                mbar_arrive(&sm.red[stage]);
            }
            bool last = false;
            int b = 0;
            if (warp == 0) {
                const uint32_t ph = (red_phase >> stage) & 1u;
                red_phase ^= 1u << stage;
                const bool ok = mbar_wait(&sm.red[stage], ph, &sm.abort_flag);
                float2 v = lane < kConsumerWarps ? sm.scratch[stage][lane] : make_float2(-INFINITY, 0.f);
                m = v.x; sum = v.y;
#pragma unroll
                for (int off = kConsumerWarps / 2; off > 0; off >>= 1) {
                    float m2 = __shfl_xor_sync(0xffffffffu, m, off);
                    float s2 = __shfl_xor_sync(0xffffffffu, sum, off);
                    merge_ms(m, sum, m2, s2, p.c);
                }
                b = mt.unit / (R * P);
                int is_last = 0;
                if (lane == 0 && ok) {
                    const int rem = mt.unit % (R * P);
                    p.partial[((size_t)b * R + rem / P) * P + rem % P] = make_float2(m, sum);
                    __threadfence();
                    is_last = atomicAdd(&p.ticket1[b], 1) == R * P - 1;
                }
                last = __shfl_sync(0xffffffffu, is_last, 0) != 0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
            if (last) {
                __threadfence();
                finalize_sequence<E>(p, b, lane);
            }
        }
    }
    if (sm.abort_flag && lane == 0) atomicOr(&p.heads[2], kDevTimeout);
}

}  // namespace ears
