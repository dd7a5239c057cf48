// Kernel 2: the token at the first rejected position, or the bonus token.
//
// For sequence b with accepted length n (written by kernel 1):
//   n < K : masses r_v = max(0, P_t(v) - P_d(v)) on rows (b, n)      (residual)
//   n = K : masses r_v = P_t(v) on the extra target row (b, K)        (bonus)
// and the token is the smallest j with u*S < C_j (C running sum, S total, u the
// 53-bit uniform of slot K).  The paper leaves this step to the target model
// (Sec. 3.1); this is the speculative-sampling rule of its refs. [1], [2].
//
// Only the one or two rows that matter are read.  They are cut into pieces that
// persistent CTAs pull from a queue and stream through shared memory like kernel 1;
// each warp reduces 512-element segments to one fp64 sum.  The CTA delivering the
// last piece of a sequence scans the segment sums, picks the segment holding u*S,
// re-reads those 512 elements and finishes the scan inside one warp.  Terms are
// fp32 exp2 of an fp32 argument; normalisation, subtraction and all sums are fp64.
#pragma once
#include "ears_k1.cuh"

namespace ears {

struct RowNorm {
    float mt, md;     // row maxima
    double izt, izd;  // 1 / Z
};

// Mass of one vocabulary entry.  Explicit rounding intrinsics so that the streaming
// pass and the final in-segment pass produce identical bits.
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

// Segment sums of one staged chunk; warp w takes segments w, w+8, ...
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
    int L = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : 0);
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

// Final pick for sequence b by one warp, after all its segment sums are in memory.
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

template <typename E, int STAGES>
__global__ void __launch_bounds__(kThreads, 2) k2_final_token(const Params p) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = PipeSmem<STAGES, 2>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts2, cpp = p.plan.cpp2, nseg = p.plan.nseg;
    const bool use_tma = p.plan.use_tma != 0;
    const int chunks_per_row = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    const long long total_units = (long long)p.B * P;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    pipe_init(sm, use_tma);

    if (warp == kConsumerWarps) {
        // ------------------------------ loader warp
        uint32_t q = 0;
        bool ok = true;
        while (ok) {
            long long u = 0;
            if (lane == 0) u = atomicAdd(&p.heads[1], 1);
            u = __shfl_sync(0xffffffffu, u, 0);
            if (u >= total_units || sm.abort_flag) break;
            const int b = (int)(u / P), part = (int)(u % P);
            const int n = p.out_len[b];
            if (n < 0) continue;  // invalid sequence: outputs already written by kernel 1
            const bool resid = n < K;
            const E* trow = reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, n, K) * V;
            const E* drow = reinterpret_cast<const E*>(p.d) + (size_t)draft_row(b, resid ? n : 0, K) * V;
            const int ch0 = part * cpp;
            const int ch1 = min(chunks_per_row, ch0 + cpp);
            for (int ch = ch0; ch < ch1; ++ch, ++q) {
                ok = loader_acquire(sm, q, lane);
                if (!ok) break;
                const int stage = q % STAGES;
                const int e0 = ch * CHUNK_ELEMS;
                const int ne = min(CHUNK_ELEMS, V - e0);
                const uint32_t bytes = (uint32_t)ne * (uint32_t)sizeof(E);
                if (lane == 0) {
                    sm.meta[stage] = StageMeta{(int)u, ne, (ch == ch0 ? 1 : 0) | (ch == ch1 - 1 ? 2 : 0), e0};
                    sm.meta_aux[stage] = n;
                }
                if (use_tma) {
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&sm.full[stage], resid ? 2 * bytes : bytes);
                        bulk_load(sm.buf[stage][0], trow + e0, bytes, &sm.full[stage]);
                        if (resid) bulk_load(sm.buf[stage][1], drow + e0, bytes, &sm.full[stage]);
                    }
                } else {
                    lane_copy<E>(sm.buf[stage][0], trow + e0, ne, lane);
                    if (resid) lane_copy<E>(sm.buf[stage][1], drow + e0, ne, lane);
                    __syncwarp();
                    mbar_arrive(&sm.full[stage]);
                }
            }
        }
        if (ok && loader_acquire(sm, q, lane)) {
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
        uint32_t red_phase = 0;
        RowNorm rn{0.f, 0.f, 0.0, 0.0};
        for (uint32_t q = 0;; ++q) {
            const int stage = q % STAGES;
            if (!mbar_wait(&sm.full[stage], (q / STAGES) & 1u, &sm.abort_flag)) break;
            const StageMeta mt = sm.meta[stage];
            if (mt.unit < 0) break;
            const int n = sm.meta_aux[stage];
            const int b = mt.unit / P;
            const bool resid = n < K;
            if (mt.flags & 1) {
                const float2 st = __ldcg(&p.rowstat[(size_t)b * R + (resid ? 2 * n : 2 * K)]);
                const float2 sd = resid ? __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]) : make_float2(0.f, 1.f);
                rn = RowNorm{st.x, sd.x, 1.0 / (double)st.y, 1.0 / (double)sd.y};
            }
            double* seg_out = p.segsum + (size_t)b * nseg + mt.elem0 / kSegElems;
            if (resid) chunk_segments<E, true>(sm.buf[stage][0], sm.buf[stage][1], mt.nelem, warp, lane, rn, p.c, seg_out);
            else chunk_segments<E, false>(sm.buf[stage][0], sm.buf[stage][0], mt.nelem, warp, lane, rn, p.c, seg_out);
            if (!(mt.flags & 2)) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[stage]);
                continue;
            }
            // last chunk of the unit: publish, count the arrival, maybe finish the sequence
            if (lane == 0) {
                __threadfence();
                mbar_arrive(&sm.red[stage]);
            }
            bool last = false;
            if (warp == 0) {
                const uint32_t ph = (red_phase >> stage) & 1u;
                red_phase ^= 1u << stage;
                const bool ok = mbar_wait(&sm.red[stage], ph, &sm.abort_flag);
                int is_last = 0;
                if (lane == 0 && ok) {
                    __threadfence();
                    is_last = atomicAdd(&p.ticket2[b], 1) == P - 1;
                }
                last = __shfl_sync(0xffffffffu, is_last, 0) != 0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
            if (last) {
                __threadfence();
                select_token<E>(p, b, n, lane);
            }
        }
    }
    if (sm.abort_flag && lane == 0) atomicOr(&p.heads[2], kDevTimeout);
}

}  // namespace ears
