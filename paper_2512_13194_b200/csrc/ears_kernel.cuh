// The verification step as one persistent kernel.
//
// Work is cut into "units" (a piece of one logits row) that CTAs pull from an atomic
// queue, sequence by sequence, so that the 2K+1 rows of a sequence stream through the
// GPU at about the same time.  Inside a CTA:
//
//   loader warp    pulls units and streams them into a ring of shared-memory slots with
//                  1-D bulk asynchronous copies completing on mbarriers (element-wise
//                  copies when the data is not 16-byte aligned);
//   8 consumer     keep a running (max, sum exp2) per thread over the slots [softmax
//   warps          statistics, Sec. 3.1], reduce them per unit and publish the piece;
//                  the CTA that delivers the last piece of a sequence hands the
//                  sequence to its epilogue warp;
//   epilogue warp  merges the pieces, forms P_t(x), P_d(x), max P_t = 1/Z_t, draws U_k,
//                  decides every position (Sec. 3.2 with the guards of Sec. 3.3 item 2),
//                  scans for the first rejection (Sec. 3.1) and asks the loader for the
//                  one or two rows the final token needs.  Those rows were streamed
//                  moments ago by this and neighbouring CTAs and are normally still in
//                  L2, so the second pass costs little or no HBM traffic.  The consumers
//                  turn them into fp64 segment sums of the masses; the epilogue warp then
//                  picks the token by inverse CDF.
//
// No CTA ever waits for another CTA; all waits inside a CTA are bounded.
#pragma once
#include "ears_common.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"

namespace ears {

enum ChunkKind : int { kStats = 0, kBonus = 1, kResid = 2, kDrain = 3, kEnd = 4 };
enum MsgKind : int { kMsgFinalize = 0, kMsgSelect = 1, kMsgDrain = 2, kMsgExit = 3, kMsgJob = 4, kMsgAck = 5 };

struct StageMeta {
    int kind;    // ChunkKind
    int id;      // unit index (statistics) or sequence index (final-token rows)
    int nelem;   // valid elements per row in the slot
    int flags;   // bit 0: first chunk of the unit / row, bit 1: last chunk
    int elem0;   // index of the slot's first element within its row
    int aux;     // accepted length n of the sequence (final-token rows)
};

struct Msg { int kind, a, b; };

// Single-producer single-consumer ring in shared memory.  One lane pushes, one lane pops.
template <int CAP>
struct Mailbox {
    volatile int head, tail;
    volatile int slot[CAP][3];

    __device__ __forceinline__ void init() { head = 0; tail = 0; }

    // false only when the block is aborting or the time limit passed
    __device__ __forceinline__ bool push(const Msg& m, volatile int* abort_flag, unsigned long long limit_ns) {
        unsigned long long t0 = 0;
        for (unsigned spin = 0; tail - head >= CAP; ++spin) {
            if ((spin & 15u) == 15u) {
                if (*abort_flag) return false;
                unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
            }
            __nanosleep(40);
        }
        const int t = tail;
        slot[t % CAP][0] = m.kind; slot[t % CAP][1] = m.a; slot[t % CAP][2] = m.b;
        __threadfence_block();
        tail = t + 1;
        return true;
    }
    __device__ __forceinline__ bool try_pop(Msg& m) {
        const int h = head;
        if (h == tail) return false;
        __threadfence_block();
        m.kind = slot[h % CAP][0]; m.a = slot[h % CAP][1]; m.b = slot[h % CAP][2];
        __threadfence_block();
        head = h + 1;
        return true;
    }
    __device__ __forceinline__ bool pop(Msg& m, volatile int* abort_flag, unsigned long long limit_ns) {
        unsigned long long t0 = 0;
        for (unsigned spin = 0;; ++spin) {
            if (try_pop(m)) return true;
            if ((spin & 15u) == 15u) {
                if (*abort_flag) return false;
                unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
            }
            __nanosleep(64);
        }
    }
};

// consumer warp 0 -> epilogue warp
constexpr int kEpiCap = 32;
// epilogue warp -> loader warp.  The loader serves this ring before it pulls a new unit, and one
// unit produces at most one entry, so at most kEpiCap + slots + 2 entries are ever outstanding:
// the ring never fills and the epilogue warp never blocks on it.
constexpr int kJobCap = 64;
constexpr unsigned long long kIdleLimitNs = 30000000000ull;  // an idle warp may wait for the whole kernel

template <int STAGES>
struct PipeSmem {
    alignas(128) unsigned char buf[STAGES][kChunkBytes];
    alignas(8) uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t red[STAGES];
    StageMeta meta[STAGES];
    float2 scratch[STAGES][kConsumerWarps];
    Mailbox<kEpiCap> epi;
    Mailbox<kJobCap> jobs;
    int abort_flag;
};

// ---- loader helpers -----------------------------------------------------------
template <int STAGES>
__device__ __forceinline__ bool loader_acquire(PipeSmem<STAGES>& sm, uint32_t q, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(&sm.empty[q % STAGES], ((q / STAGES) & 1u) ^ 1u, &sm.abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

template <typename E>
__device__ __forceinline__ void lane_copy(void* dst, const E* src, int n, int lane) {
    E* o = reinterpret_cast<E*>(dst);
    for (int i = lane; i < n; i += 32) o[i] = __ldg(src + i);
}

// After an abort: give copies that may still be in flight a bounded time to land
// before the CTA's shared memory is released.
template <int STAGES>
__device__ __forceinline__ void loader_drain(PipeSmem<STAGES>& sm, uint32_t issued) {
    uint32_t first = issued > STAGES ? issued - STAGES : 0;
    for (uint32_t q = first; q < issued; ++q) {
        unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(&sm.full[q % STAGES], (q / STAGES) & 1u)) {
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
    }
}

// Publishes a slot: `nelem` elements from src0 (and, at the half-slot offset, from src1).
template <typename E, int STAGES>
__device__ __forceinline__ void loader_fill(PipeSmem<STAGES>& sm, int stage, const StageMeta& mt, bool use_tma,
                                            const E* src0, const E* src1, int lane) {
    if (lane == 0) sm.meta[stage] = mt;
    const uint32_t bytes = (uint32_t)mt.nelem * (uint32_t)sizeof(E);
    if (use_tma) {
        if (lane == 0) {
            if (bytes == 0 || !src0) {
                mbar_arrive(&sm.full[stage]);
            } else {
                mbar_arrive_expect_tx(&sm.full[stage], src1 ? 2 * bytes : bytes);
                bulk_load(sm.buf[stage], src0, bytes, &sm.full[stage]);
                if (src1) bulk_load(sm.buf[stage] + kChunkBytes / 2, src1, bytes, &sm.full[stage]);
            }
        }
    } else {
        if (src0) lane_copy<E>(sm.buf[stage], src0, mt.nelem, lane);
        if (src1) lane_copy<E>(sm.buf[stage] + kChunkBytes / 2, src1, mt.nelem, lane);
        __syncwarp();
        mbar_arrive(&sm.full[stage]);
    }
}

// ---- consumer arithmetic --------------------------------------------------------
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

struct RowNorm {
    float mt, md;     // row maxima
    double izt, izd;  // 1 / Z
};

// Mass of one vocabulary entry for the final draw: P_t(v), or max(0, P_t(v) - P_d(v)).
// Explicit rounding intrinsics so that the streaming pass and the in-segment pass
// produce identical bits.
template <bool RESID>
__device__ __forceinline__ double entry_mass(float xt, float xd, const RowNorm& rn, float c) {
    const float et = ex2_approx(__fmul_rn(__fsub_rn(xt, rn.mt), c));
    double r = __dmul_rn((double)et, rn.izt);
    if (RESID) {
        const float ed = ex2_approx(__fmul_rn(__fsub_rn(xd, rn.md), c));
        r = fmax(__dsub_rn(r, __dmul_rn((double)ed, rn.izd)), 0.0);
    }
    return r;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

__device__ __forceinline__ double warp_inclusive_scan(double v, int lane) {
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    return v;
}

// fp64 sums of kSegElems-element segments of a staged chunk; warp w takes segments w, w+8, ...
template <typename E, bool RESID>
__device__ __forceinline__ void chunk_segments(const unsigned char* bt, const unsigned char* bd, int nelem,
                                               int warp, int lane, const RowNorm& rn, float c, double* seg_out) {
    constexpr int N = Vec<E>::N;
    constexpr int VECS = kSegElems / (32 * N);  // 16-byte vectors per lane per segment
    const int nseg = (nelem + kSegElems - 1) / kSegElems;
    for (int sgm = warp; sgm < nseg; sgm += kConsumerWarps) {
        double acc = 0.0;
#pragma unroll
        for (int j = 0; j < VECS; ++j) {
            const int vec = sgm * (kSegElems / N) + j * 32 + lane;
            float xt[N], xd[N];
            Vec<E>::load(bt, vec, xt);
            if (RESID) Vec<E>::load(bd, vec, xd);
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const double r = entry_mass<RESID>(xt[i], RESID ? xd[i] : 0.f, rn, c);
                if (vec * N + i < nelem) acc += r;
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) seg_out[sgm] = acc;
    }
}

// ---- epilogue warp: decisions -----------------------------------------------------
// Merges the pieces of all 2K+1 rows, writes (m, Z) per row, decides every position
// (Sec. 3.2 steps 1-5 with the guards of Sec. 3.3 item 2) and writes the accepted
// prefix (Sec. 3.1).  Returns the accepted length n, or -1 for an invalid sequence.
template <typename E>
__device__ int finalize_sequence(const Params& p, int b, int lane) {
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
        return -1;
    }
    for (int j = lane; j <= K; j += 32) ot[j] = j < first_reject ? p.x[(size_t)b * K + j] : -1;
    if (lane == 0) p.out_len[b] = first_reject;
    return first_reject;
}

// ---- epilogue warp: final token ---------------------------------------------------
// Slow whole-row draw from P_t by one warp (used only if a residual has no mass).
template <typename E>
__device__ int warp_sample_pt_slow(const E* row, int V, const RowNorm& rn, float c, double u, int lane, double* S_out) {
    const int per = (V + 31) / 32;
    const int v0 = min(V, lane * per), v1 = min(V, v0 + per);
    double loc = 0.0;
    for (int v = v0; v < v1; ++v) loc += entry_mass<false>(load_logit(row + v), 0.f, rn, c);
    const double inc = warp_inclusive_scan(loc, lane);
    const double S = __shfl_sync(0xffffffffu, inc, 31);
    const double target = u * S;
    const unsigned hit = __ballot_sync(0xffffffffu, target < inc && loc > 0.0);
    const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
    const int L = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : 0);
    int tok = -1;
    if (lane == L) {
        double cum = inc - loc;
        int lastpos = -1;
        for (int v = v0; v < v1; ++v) {
            const double r = entry_mass<false>(load_logit(row + v), 0.f, rn, c);
            if (r > 0.0) lastpos = v;
            cum += r;
            if (target < cum && r > 0.0) { tok = v; break; }
        }
        if (tok < 0) tok = lastpos;
    }
    *S_out = S;
    return __shfl_sync(0xffffffffu, tok, L);
}

// Inverse-CDF pick for sequence b (accepted length n) from its segment sums:
// token = smallest j with u*S < C_j.  Level 1 finds the segment, level 2 re-reads its
// kSegElems entries and finishes inside the warp.
template <typename E>
__device__ void select_token(const Params& p, int b, int n, int lane) {
    const int K = p.K, V = p.V, R = 2 * K + 1, nseg = p.plan.nseg;
    const bool resid = n < K;
    const E* trow = reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, n, K) * V;
    const E* drow = reinterpret_cast<const E*>(p.d) + (size_t)draft_row(b, resid ? n : 0, K) * V;
    const float2 st = __ldcg(&p.rowstat[(size_t)b * R + (resid ? 2 * n : 2 * K)]);
    const float2 sd = resid ? __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]) : make_float2(0.f, 1.f);
    const RowNorm rn{st.x, sd.x, 1.0 / (double)st.y, 1.0 / (double)sd.y};
    const double* ss = p.segsum + (size_t)b * nseg;
    const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)K);

    // level 1: which segment
    const int per = (nseg + 31) / 32;
    const int g0 = min(nseg, lane * per), g1 = min(nseg, g0 + per);
    double loc = 0.0;
    for (int g = g0; g < g1; ++g) loc += __ldcg(ss + g);
    const double inc = warp_inclusive_scan(loc, lane);
    const double S = __shfl_sync(0xffffffffu, inc, 31);
    int tok;
    double S_used = S;
    if (!(S >= kTinyMass)) {
        // a rejection implies residual mass; if rounding erased it, draw from P_t instead
        tok = warp_sample_pt_slow<E>(trow, V, rn, p.c, u, lane, &S_used);
    } else {
        const double target = u * S;
        const unsigned hit = __ballot_sync(0xffffffffu, target < inc && loc > 0.0);
        const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
        const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
        const double excl_L = __shfl_sync(0xffffffffu, inc - loc, L);
        const int gl0 = __shfl_sync(0xffffffffu, g0, L), gl1 = __shfl_sync(0xffffffffu, g1, L);
        int seg = -1, lastseg = gl0;
        double before = excl_L, before_last = excl_L;
        {
            double cum = excl_L;
            for (int g = gl0; g < gl1; ++g) {  // every lane walks the same few sums
                const double v = __ldcg(ss + g);
                if (v > 0.0) { lastseg = g; before_last = cum; }
                if (seg < 0 && v > 0.0 && target < cum + v) { seg = g; before = cum; }
                cum += v;
            }
        }
        if (seg < 0) { seg = lastseg; before = before_last; }
        // level 2: which element of the segment
        const double tin = target - before;
        constexpr int N = Vec<E>::N;
        const int base = seg * kSegElems;
        double run = 0.0;
        int found = -1, lastpos = -1;
        for (int j = 0; j < kSegElems / (32 * N) && found < 0; ++j) {
            const int e0 = base + (j * 32 + lane) * N;
            double r[N], mine = 0.0;
            int mylast = -1;
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const int e = e0 + i;
                r[i] = 0.0;
                if (e < V) {
                    const float xt = load_logit(trow + e);
                    const float xd = resid ? load_logit(drow + e) : 0.f;
                    r[i] = resid ? entry_mass<true>(xt, xd, rn, p.c) : entry_mass<false>(xt, 0.f, rn, p.c);
                }
                if (r[i] > 0.0) mylast = e;
                mine += r[i];
            }
            const double incl = warp_inclusive_scan(mine, lane);
            const unsigned h = __ballot_sync(0xffffffffu, tin < run + incl && mine > 0.0);
            // remember the last positive entry seen so far (fallback if rounding hides the hit)
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mylast = max(mylast, __shfl_xor_sync(0xffffffffu, mylast, off));
            if (h) {
                const int Lh = __ffs(h) - 1;
                int t_here = -1;
                if (lane == Lh) {
                    double cum = run + (incl - mine);
                    int lp = -1;
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        cum += r[i];
                        if (r[i] > 0.0) lp = e0 + i;
                        if (t_here < 0 && r[i] > 0.0 && tin < cum) t_here = e0 + i;
                    }
                    if (t_here < 0) t_here = lp;
                }
                found = __shfl_sync(0xffffffffu, t_here, Lh);
            } else {
                lastpos = max(lastpos, mylast);
                run += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        tok = found >= 0 ? found : lastpos;
    }
    if (lane == 0) {
        p.out_tok[(size_t)b * (K + 1) + n] = tok;
        p.resid[b] = S_used;
    }
}

// ---- the kernel -------------------------------------------------------------------
template <typename E, int STAGES>
__global__ void __launch_bounds__(kThreads, 2) ears_verify_kernel(const Params p) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = PipeSmem<STAGES>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1, cpp = p.plan.cpp1, nseg = p.plan.nseg;
    const bool use_tma = p.plan.use_tma != 0;
    const int chunks_per_row = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    const long long total_units = (long long)p.B * R * P;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const E* tbase = reinterpret_cast<const E*>(p.t);
    const E* dbase = reinterpret_cast<const E*>(p.d);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm.full[s], use_tma ? 1u : 32u);
            mbar_init(&sm.empty[s], kConsumerWarps);
            mbar_init(&sm.red[s], kConsumerWarps);
        }
        sm.epi.init();
        sm.jobs.init();
        sm.abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();

    if (warp == kLoaderWarp) {
        // =============================== loader warp
        uint32_t q = 0;
        bool ok = true, stats_done = false, acked = false;
        while (ok && !acked) {
            // 1. rows for a final token come first: they are hot in L2 right now
            Msg job{-1, 0, 0};
            int have = 0;
            if (lane == 0) {
                if (stats_done) have = sm.jobs.pop(job, &sm.abort_flag, kIdleLimitNs) ? 1 : -1;
                else have = sm.jobs.try_pop(job) ? 1 : 0;
            }
            have = __shfl_sync(0xffffffffu, have, 0);
            if (have < 0) { ok = false; break; }
            if (have > 0) {
                job.kind = __shfl_sync(0xffffffffu, job.kind, 0);
                job.a = __shfl_sync(0xffffffffu, job.a, 0);
                job.b = __shfl_sync(0xffffffffu, job.b, 0);
                if (job.kind == kMsgAck) { acked = true; break; }
                const int b = job.a, n = job.b;
                const bool resid = n < K;
                const int step = resid ? CHUNK_ELEMS / 2 : CHUNK_ELEMS;
                const E* trow = tbase + (size_t)target_row(b, n, K) * V;
                const E* drow = resid ? dbase + (size_t)draft_row(b, n, K) * V : nullptr;
                for (int e0 = 0; e0 < V; e0 += step, ++q) {
                    ok = loader_acquire(sm, q, lane);
                    if (!ok) break;
                    const int ne = min(step, V - e0);
                    const StageMeta mt{resid ? kResid : kBonus, b, ne, (e0 == 0 ? 1 : 0) | (e0 + step >= V ? 2 : 0), e0, n};
                    loader_fill<E>(sm, q % STAGES, mt, use_tma, trow + e0, resid ? drow + e0 : nullptr, lane);
                }
                continue;
            }
            // 2. next piece of a row for the statistics pass
            long long u = 0;
            if (lane == 0) u = atomicAdd(&p.heads[0], 1);
            u = __shfl_sync(0xffffffffu, u, 0);
            if (sm.abort_flag) { ok = false; break; }
            if (u >= total_units) {
                // nothing left to pull: tell the consumers, then serve final-token rows until acknowledged
                ok = loader_acquire(sm, q, lane);
                if (!ok) break;
                loader_fill<E>(sm, q % STAGES, StageMeta{kDrain, 0, 0, 0, 0, 0}, use_tma, nullptr, nullptr, lane);
                ++q;
                stats_done = true;
                continue;
            }
            const int b = (int)(u / (R * P));
            const int rem = (int)(u % (R * P));
            const int ridx = rem / P, part = rem % P;
            const E* row = (ridx == 2 * K) ? tbase + (size_t)target_row(b, K, K) * V
                                           : ((ridx & 1) ? dbase + (size_t)draft_row(b, ridx >> 1, K) * V
                                                         : tbase + (size_t)target_row(b, ridx >> 1, K) * V);
            const int ch0 = part * cpp;
            const int ch1 = min(chunks_per_row, ch0 + cpp);
            for (int ch = ch0; ch < ch1; ++ch, ++q) {
                ok = loader_acquire(sm, q, lane);
                if (!ok) break;
                const int e0 = ch * CHUNK_ELEMS;
                const StageMeta mt{kStats, (int)u, min(CHUNK_ELEMS, V - e0), (ch == ch0 ? 1 : 0) | (ch == ch1 - 1 ? 2 : 0), e0, 0};
                loader_fill<E>(sm, q % STAGES, mt, use_tma, row + e0, nullptr, lane);
            }
        }
        if (ok && loader_acquire(sm, q, lane)) {
            loader_fill<E>(sm, q % STAGES, StageMeta{kEnd, 0, 0, 0, 0, 0}, use_tma, nullptr, nullptr, lane);
        } else if (use_tma && lane == 0) {
            loader_drain(sm, q);
        }
    } else if (warp == kEpilogueWarp) {
        // =============================== epilogue warp
        for (;;) {
            Msg m{kMsgExit, 0, 0};
            int got = 0;
            if (lane == 0) got = sm.epi.pop(m, &sm.abort_flag, kIdleLimitNs) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) break;
            m.kind = __shfl_sync(0xffffffffu, m.kind, 0);
            m.a = __shfl_sync(0xffffffffu, m.a, 0);
            m.b = __shfl_sync(0xffffffffu, m.b, 0);
            if (m.kind == kMsgExit) break;
            if (m.kind == kMsgFinalize) {
                __threadfence();
                const int n = finalize_sequence<E>(p, m.a, lane);
                if (n >= 0) {
                    __threadfence();  // row statistics must be visible to the consumers of the job
                    __syncwarp();
                    int pushed = 1;
                    if (lane == 0) pushed = sm.jobs.push(Msg{kMsgJob, m.a, n}, &sm.abort_flag, kWaitLimitNs) ? 1 : 0;
                    if (!__shfl_sync(0xffffffffu, pushed, 0)) break;
                }
            } else if (m.kind == kMsgSelect) {
                __threadfence();
                select_token<E>(p, m.a, m.b, lane);
            } else if (m.kind == kMsgDrain) {
                int pushed = 1;
                if (lane == 0) pushed = sm.jobs.push(Msg{kMsgAck, 0, 0}, &sm.abort_flag, kWaitLimitNs) ? 1 : 0;
                if (!__shfl_sync(0xffffffffu, pushed, 0)) break;
            }
        }
    } else {
        // =============================== consumer warps
        const int tid = threadIdx.x;
        float m_run = -INFINITY;
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t red_phase = 0;
        RowNorm rn{0.f, 0.f, 0.0, 0.0};
        for (uint32_t q = 0;; ++q) {
            const int stage = q % STAGES;
            if (!mbar_wait(&sm.full[stage], (q / STAGES) & 1u, &sm.abort_flag)) break;
            const StageMeta mt = sm.meta[stage];
            if (mt.kind == kEnd) {
                if (warp == 0 && lane == 0) sm.epi.push(Msg{kMsgExit, 0, 0}, &sm.abort_flag, kWaitLimitNs);
                break;
            }
            if (mt.kind == kDrain) {
                if (warp == 0 && lane == 0) sm.epi.push(Msg{kMsgDrain, 0, 0}, &sm.abort_flag, kWaitLimitNs);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[stage]);
                continue;
            }
            if (mt.kind == kStats) {
                if (mt.flags & 1) { m_run = -INFINITY; s[0] = s[1] = s[2] = s[3] = 0.f; }
                chunk_stats<E>(sm.buf[stage], mt.nelem, tid, p.c, m_run, s);
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
                    if (lane == 0 && ok) {
                        const int b = mt.id / (R * P);
                        const int rem = mt.id % (R * P);
                        p.partial[((size_t)b * R + rem / P) * P + rem % P] = make_float2(m, sum);
                        __threadfence();
                        if (atomicAdd(&p.ticket1[b], 1) == R * P - 1)  // last piece of the sequence
                            sm.epi.push(Msg{kMsgFinalize, b, 0}, &sm.abort_flag, kWaitLimitNs);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[stage]);
                continue;
            }
            // rows of a final token: fp64 segment sums of the masses
            const int b = mt.id, n = mt.aux;
            const bool resid = mt.kind == kResid;
            if (mt.flags & 1) {
                const float2 st = __ldcg(&p.rowstat[(size_t)b * R + (resid ? 2 * n : 2 * K)]);
                const float2 sd = resid ? __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]) : make_float2(0.f, 1.f);
                rn = RowNorm{st.x, sd.x, 1.0 / (double)st.y, 1.0 / (double)sd.y};
            }
            double* seg_out = p.segsum + (size_t)b * nseg + mt.elem0 / kSegElems;
            if (resid) chunk_segments<E, true>(sm.buf[stage], sm.buf[stage] + kChunkBytes / 2, mt.nelem, warp, lane, rn, p.c, seg_out);
            else chunk_segments<E, false>(sm.buf[stage], sm.buf[stage], mt.nelem, warp, lane, rn, p.c, seg_out);
            if (mt.flags & 2) {
                // last chunk of the row(s): publish the sums, then hand the pick to the epilogue warp
                if (lane == 0) {
                    __threadfence();
                    mbar_arrive(&sm.red[stage]);
                }
                if (warp == 0) {
                    const uint32_t ph = (red_phase >> stage) & 1u;
                    red_phase ^= 1u << stage;
                    const bool ok = mbar_wait(&sm.red[stage], ph, &sm.abort_flag);
                    if (lane == 0 && ok) sm.epi.push(Msg{kMsgSelect, b, n}, &sm.abort_flag, kWaitLimitNs);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
        }
    }
    if (sm.abort_flag && lane == 0) atomicOr(&p.heads[2], kDevTimeout);
}

}  // namespace ears
