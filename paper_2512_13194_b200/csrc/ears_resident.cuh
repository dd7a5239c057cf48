// The verification step with the rows of one position resident in shared memory.
//
// Work item = one position of one sequence: the pair (target row k, draft row k), or the
// extra target row K.  A thread-block cluster of C CTAs takes an item; CTA j brings the j-th
// slice of the row(s) into its own shared memory with 1-D bulk asynchronous copies (each
// CTA fetches for itself; element-wise copies when the rows are not 16-byte aligned) and everything else
// is computed from there, so that every logit crosses HBM exactly once:
//
//   1. softmax statistics (max, sum exp2) of the slices while the copies land [Sec. 3.1];
//   2. the C partial results are exchanged through distributed shared memory (remote stores
//      plus a remote mbarrier arrive per peer) and every CTA forms the rows' (max, Z);
//   3. every CTA takes the decision of Sec. 3.2 (with the guards of Sec. 3.3 item 2) for the
//      position -- redundantly, from identical numbers, hence identically;
//   4. a rejected position draws its replacement token at once from max(0, P_t - P_d) of the
//      resident slices ("as if this were the first rejection"); the extra row K always draws
//      its bonus token from P_t.  Segment sums per CTA, totals exchanged through distributed
//      shared memory, and the one CTA that holds u*S picks the entry;
//   5. the last item of a sequence to finish (an atomic ticket) scans the K decisions for the
//      first rejection [Sec. 3.1] and writes the outputs.
//
// No CTA ever waits for work another cluster has yet to start; the only waits are on copies
// into the CTA's own memory and on the C peers of its own cluster, all bounded in time.
#pragma once
#include "ears_common.cuh"
#include "ears_math.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"

namespace ears {

constexpr int kRWarps = 8;
constexpr int kRThreads = kRWarps * 32;
constexpr int kRSubBytes = 8192;          // bytes of each row that one copy barrier covers
constexpr int kRMaxSub = 16;              // copy barriers per CTA: a slice holds <= 128 KB of each row
constexpr int kRMaxCluster = 16;
constexpr int kRMaxSeg = kRMaxSub * kRSubBytes / 2 / kSegElems;  // segment sums of the largest slice (2-byte elements)

struct RParams {
    const void* t;
    const void* d;
    const int32_t* x;
    int B, K, V;
    float c;              // log2(e) / temperature
    double T, beta;
    const float* seq_T;   // [B] per-sequence temperature, or NULL
    const float* seq_beta;  // [B] per-sequence beta, or NULL
    unsigned long long seed, offset;
    long long b_first;
    int32_t* out_len;
    int32_t* out_tok;
    double* pt_tok;
    double* pd_tok;
    double* max_pt;
    uint8_t* cls;
    double* resid;
    int* heads;           // [0] item queue, [1] finished sequences, [2] status word, [3] published jobs, [4] piece tickets given out ([1], [3], [4]: streaming clusters)
    int* ticket;          // [B] items of the sequence that are done
    signed char* flag;    // [B,K+1] 1 accepted directly / row usable, 2 accepted by pardon, 0 rejected, -1 invalid
    int32_t* cand;        // [B,K+1] token drawn at the position (rejected positions and slot K)
    double* cand_mass;    // [B,K+1] mass that token was drawn from
    float4* rowstat;      // [B,K+1] (max, Z) of the item's target and draft rows (streaming clusters only)
    unsigned long long* seqmask;  // [B] positions decided (low word) and accepted (high word), K <= 30 (streaming clusters only)
    // second-pass jobs of the streaming clusters (a sequence's first rejected position), served by every CTA:
    unsigned long long* ready;    // [B] published jobs in the order of heads[3]: (b + 1) << 32 | n
    int* ticket2;                 // [B] pieces of the sequence's job that are done
    double* segsums;              // [B, nseg] masses per kSegElems entries of the job's rows
    int nseg, job_elems, parts2;  // segments per row; entries per piece; pieces per job
    int unc_entropy;      // 1: the tolerance is scaled by H(P_t) / ln V instead of 1 - max P_t [Sec. 5 item 1]
    double* entropy;      // [B,K] H(P_t) of every target row, or NULL; the entropy kernels (ENT) fill it
    int C;                // CTAs per cluster
    int slice;            // elements of a row per CTA, a multiple of kSegElems
    int buf_bytes;        // shared-memory bytes reserved per row slice (slice bytes rounded up to kRSubBytes)
    int use_tma;
    int n_clusters;
    int want_stats;       // the caller asked for P_t(x), P_d(x), max P_t or the class of every position
    int* zero_ptr;        // counter block of the next call, cleared by this kernel (zero_words ints; may be 0)
    int zero_words;
    int ordered;          // 1: a cluster takes a whole sequence, position by position, and stops at its first
                          //    rejection [Sec. 3.1]: later rows are never read
};

struct RSmem {
    alignas(8) uint64_t full[kRMaxSub];
    uint64_t xbar[2];                    // statistics exchange, alternating by round
    uint64_t mbar2[2];                   // mass-total exchange, alternating by mass round
    alignas(16) float4 xstat[2][kRMaxCluster * kRWarps];   // (m_t, s_t, m_d, s_d) of every warp of every peer
    float xw[2][kRMaxCluster * kRWarps]; // sum e t of the target slice of every warp of every peer (entropy kernels)
    double xmass[2][kRMaxCluster];       // mass totals of every peer
    int xnext[2];                        // next item of the cluster (written by rank 0)
    double segsum[kRMaxSeg];
    float2 rs_t, rs_d;                   // (max, Z) of the item's rows
    int dec;                             // decision broadcast: 1 accept, 0 reject, -1 invalid
    int pick_rank;                       // CTA that holds u*S (-1: no mass anywhere)
    double pick_tin, pick_S;
    int abort_flag;
};

// ---- cluster primitives (sm_90+) ------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_peer(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void peer_store(uint32_t addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ void peer_store(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void peer_store(uint32_t addr, int v) {
    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// Arrival on a peer's barrier; what this thread stored before is visible to whoever then
// observes the phase with cluster-scope acquire.
__device__ __forceinline__ void peer_arrive(uint32_t bar_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}
// A waiter suspended on a barrier that peers complete by remote arrivals was seen to sleep out
// its whole time hint, so the hint is kept short here and the wait polls.
constexpr unsigned kPeerWaitHintNs = 200;
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kPeerWaitHintNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
        }
    }
}
// All threads of all CTAs of the cluster.  Used at the start (barriers initialised before any
// peer arrives on them) and at the end (no CTA leaves while a peer may still store into it);
// every path to it is bounded in time.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Sub-chunk q of a slice of n valid entries: every thread takes two 16-byte vectors.
template <typename E, bool ENT>
__device__ __forceinline__ void stats_sub(const unsigned char* buf, int q, int n, int tid, float c, RowAccT<ENT>& a) {
    constexpr int SUB_VECS = kRSubBytes / 16;
    const int v0 = q * SUB_VECS + tid, v1 = v0 + kRThreads;
    stats_two_vectors<E, ENT>(buf, v0, v1, (q + 1) * SUB_VECS * Vec<E>::N <= n, n, c, a);
}

__device__ __forceinline__ void peer_store(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Warp 0 of every CTA after the exchange: the C x 8 partial results -> the rows' (max, Z) and, ENT, the
// target row's sum e t.  Lane i takes entries i, i + 32, ...: the same in every CTA, hence identical bits.
template <bool ENT>
__device__ __forceinline__ void merge_exchanged(const float4* xs, const float* xw, int parts, float cb, int lane,
                                                float& mt, float& zt, float& md, float& zd, float& wt) {
    mt = -INFINITY; md = -INFINITY;
    for (int i = lane; i < parts; i += 32) {
        mt = fmaxf(mt, xs[i].x);
        md = fmaxf(md, xs[i].z);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, off));
        md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, off));
    }
    zt = 0.f; zd = 0.f; wt = 0.f;
    for (int i = lane; i < parts; i += 32) {
        const float4 v = xs[i];
        if (ENT) {
            const float2 sw = rebase_sum_w(v.x, v.y, xw[i], mt, cb);
            zt += sw.x;
            wt += sw.y;
        } else {
            zt += rebase_sum(v.x, v.y, mt, cb);
        }
        zd += rebase_sum(v.z, v.w, md, cb);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        zt += __shfl_xor_sync(0xffffffffu, zt, off);
        zd += __shfl_xor_sync(0xffffffffu, zd, off);
        if (ENT) wt += __shfl_xor_sync(0xffffffffu, wt, off);
    }
}

// Lane 0 of warp 0 of every CTA: the decision of one position from the rows' statistics (the same
// arithmetic on the same numbers in every CTA of the cluster).  fp32 first; it stands unless R comes
// close to the threshold (the band is some 25 times the fp32 error), the caller wants the
// probabilities, or the entropy scales the tolerance: then fp64 (decide_position).
// -> the class of Sec. 3.2 step 5: 1 direct accept (R >= U), 2 pardon, 0 reject.
// `report`: this CTA writes the optional per-position outputs.
template <bool ENT, class P>
__device__ __forceinline__ int cluster_decide(const P& p, int b, int j, float lt, float ld, double U, float2 rs_t, float2 rs_d,
                                              float wt, float cb, double Tb, double betab, bool report) {
    const int K = p.K;
    double unc = -1.0, H = 0.0;
    if (ENT) {
        H = row_entropy(rs_t.y, wt);
        if (p.unc_entropy) unc = entropy_uncertainty(H, p.V);
        if (report && p.entropy) p.entropy[(size_t)b * K + j] = H;
    }
    const float pt32 = ex2_approx((lt - rs_t.x) * cb) / rs_t.y;
    const float pd32 = ex2_approx((ld - rs_d.x) * cb) / rs_d.y;
    const float ratio32 = pt32 / fmaxf(pd32, (float)kEps);
    const float unc32 = unc >= 0.0 ? (float)unc : 1.0f - 1.0f / rs_t.y;
    const float thr32 = fmaxf((float)U - (float)betab * unc32, 0.0f);
    const float diff = ratio32 - thr32;
    if (!p.want_stats && fabsf(diff) > 1e-4f * (ratio32 + thr32) + 1e-6f) return diff > 0.0f ? (ratio32 >= (float)U ? 1 : 2) : 0;
    const Decision dc = decide_position((double)lt, (double)ld, rs_t, rs_d, Tb, betab, U, unc);
    if (report && p.want_stats) {
        const size_t i = (size_t)b * K + j;
        p.pt_tok[i] = dc.pt;
        p.pd_tok[i] = dc.pd;
        p.max_pt[i] = dc.maxp;
        p.cls[i] = (uint8_t)dc.cls;
    }
    return dc.cls;
}

// ---- masses of a slice ------------------------------------------------------------
// Sums of kSegElems-entry segments of the resident slice(s); warp w takes segments w, w+8, ...
// A lane adds its few masses in fp32; lanes are added in fp64.
template <typename E, bool RESID>
__device__ __forceinline__ void slice_segments(const unsigned char* bt, const unsigned char* bd, int n, int warp, int lane,
                                               const RowNorm& rn, float c, double* segsum) {
    constexpr int N = Vec<E>::N;
    constexpr int VECS = kSegElems / (32 * N);
    const int nseg = (n + kSegElems - 1) / kSegElems;
    for (int g0 = warp; g0 < nseg; g0 += 2 * kRWarps) {  // two segments at a time: their chains overlap
        double acc[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int g = g0 + h * kRWarps;
            float a = 0.0f;
            if (g < nseg) {
#pragma unroll
                for (int j = 0; j < VECS; ++j) {
                    const int vec = g * (kSegElems / N) + j * 32 + lane;
                    float xt[N], xd[N];
                    Vec<E>::load(bt, vec, xt);
                    if (RESID) Vec<E>::load(bd, vec, xd);
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        const float r = entry_mass<RESID>(xt[i], RESID ? xd[i] : 0.f, rn, c);
                        if (vec * N + i < n) a += r;
                    }
                }
            }
            acc[h] = (double)a;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
            acc[1] += __shfl_xor_sync(0xffffffffu, acc[1], off);
        }
        if (lane == 0) {
            segsum[g0] = acc[0];
            if (g0 + kRWarps < nseg) segsum[g0 + kRWarps] = acc[1];
        }
    }
}

// Entry of segment [base, base + count) of the resident slice whose running mass first exceeds
// tin (fp64, entry order); the masses are recomputed with the bits of slice_segments.  If
// rounding hides the crossing the last entry with mass is taken; -1 if the segment has none.
template <typename E>
__device__ int pick_in_segment(const unsigned char* bt, const unsigned char* bd, bool resid, const RowNorm& rn, float c,
                               int base, int count, double tin, int lane) {
    constexpr int N = Vec<E>::N;
    constexpr int ROUNDS = kSegElems / (32 * N);
    float mass[ROUNDS][N];
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
        const int vec = base / N + j * 32 + lane;
        float xt[N], xd[N];
        Vec<E>::load(bt, vec, xt);
        Vec<E>::load(bd, vec, xd);   // bd = bt when there is no draft slice
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const bool valid = (j * 32 + lane) * N + i < count;
            mass[j][i] = !valid ? 0.f : (resid ? entry_mass<true>(xt[i], xd[i], rn, c) : entry_mass<false>(xt[i], 0.f, rn, c));
        }
    }
    double run = 0.0;
    int found = -1, lastpos = -1;
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
        if (found >= 0) break;
        const int e0 = base + (j * 32 + lane) * N;
        double mine = 0.0;
        int mylast = -1;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            if (mass[j][i] > 0.f) mylast = e0 + i;
            mine += (double)mass[j][i];
        }
        const double incl = warp_inclusive_scan(mine, lane);
        const unsigned h = __ballot_sync(0xffffffffu, tin < run + incl && mine > 0.0);
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
                    cum += (double)mass[j][i];
                    if (mass[j][i] > 0.f) lp = e0 + i;
                    if (t_here < 0 && mass[j][i] > 0.f && tin < cum) t_here = e0 + i;
                }
                if (t_here < 0) t_here = lp;
            }
            found = __shfl_sync(0xffffffffu, t_here, Lh);
        } else {
            lastpos = max(lastpos, mylast);
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    return found >= 0 ? found : lastpos;
}

// ---- end of a sequence --------------------------------------------------------------
// Called by one warp once all K+1 items of sequence b are in: first rejection [Sec. 3.1],
// accepted prefix, the token drawn at that position (or the bonus token), padding.
__device__ void finish_sequence(const RParams& p, int b, int lane) {
    const int K = p.K;
    const signed char* fl = p.flag + (size_t)b * (K + 1);
    int first_reject = K;
    bool bad = false;
    for (int k0 = 0; k0 <= K; k0 += 32) {
        const int k = k0 + lane;
        int f = 1;
        if (k <= K) f = *reinterpret_cast<const volatile signed char*>(fl + k);
        if (f < 0) bad = true;
        const unsigned rej = __ballot_sync(0xffffffffu, k < K && f == 0);
        if (rej != 0 && first_reject == K) first_reject = k0 + __ffs(rej) - 1;
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
    const int n = first_reject;
    count_decisions(p.heads, min(n + 1, K), lane, [fl](int k) { return (int)*reinterpret_cast<const volatile signed char*>(fl + k); });
    for (int j = lane; j <= K; j += 32) {
        int v = -1;
        if (j < n) v = p.x[(size_t)b * K + j];
        else if (j == n) v = __ldcg(p.cand + (size_t)b * (K + 1) + n);
        ot[j] = v;
    }
    if (lane == 0) {
        p.out_len[b] = n;
        p.resid[b] = __ldcg(p.cand_mass + (size_t)b * (K + 1) + n);
    }
}

// ---- the kernel -----------------------------------------------------------------------
template <typename E, bool ENT>
__global__ void __launch_bounds__(kRThreads, 3) ears_resident_kernel(const RParams p) {
    extern __shared__ unsigned char smem_raw[];
    RSmem& sm = *reinterpret_cast<RSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    unsigned char* buf_t = reinterpret_cast<unsigned char*>(&sm) + ((sizeof(RSmem) + 127) & ~size_t(127));
    unsigned char* buf_d = buf_t + p.buf_bytes;
    constexpr int SUB_ELEMS = kRSubBytes / (int)sizeof(E);
    const int K = p.K, V = p.V, C = p.C;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / C;
    const bool ordered = p.ordered != 0;
    // queue entries: positions (b, j) in sequence-major order, or whole sequences when ordered
    const long long n_items = ordered ? (long long)p.B : (long long)p.B * (K + 1);
    const bool use_tma = p.use_tma != 0;
    const E* tbase = reinterpret_cast<const E*>(p.t);
    const E* dbase = reinterpret_cast<const E*>(p.d);

    clear_next_counters(p);
    if (tid == 0) {
        for (int q = 0; q < kRMaxSub; ++q) mbar_init(&sm.full[q], 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&sm.xbar[i], (unsigned)(C * kRWarps)); mbar_init(&sm.mbar2[i], (unsigned)C); }
        sm.abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const int e0 = rank * p.slice;                         // this CTA's slice of every row
    const int n = max(0, min(p.slice, V - e0));
    const int nsub = (n + SUB_ELEMS - 1) / SUB_ELEMS;
    uint32_t full_phase = 0;     // bit q: parity of full[q]'s next phase
    uint32_t issued = 0;         // bit q: a copy of the current item is (or was) in flight on full[q]
    int round = 0, mround = 0;   // exchanges so far (the same in every CTA of the cluster)
    bool failed = false;
    // State of the item in hand; its copies are issued one step ahead (see the end of the loop).
    long long item = cluster_id;
    int b = 0, j = 0;
    bool pair = false;
    int next_item = 0;
    float lt = 0.f, ld = 0.f;     // the token's logits, fetched at issue time, used after the exchange
    double U = 0.0;
    bool tok_ok = true;

    // Brings in the slices of position j of sequence b and (thread 0) fetches what its decision needs.
    auto issue_item = [&](int nb, int nj) {
        b = nb;
        j = nj;
        pair = j < K;
        const E* trow = tbase + (size_t)target_row(b, j, K) * V + e0;
        const E* drow = dbase + (size_t)draft_row(b, pair ? j : 0, K) * V + e0;
        if (use_tma) {
            if (tid == 0) {
                for (int q = 0; q < nsub; ++q) {
                    const uint32_t bytes = (uint32_t)min(SUB_ELEMS, n - q * SUB_ELEMS) * (uint32_t)sizeof(E);
                    mbar_arrive_expect_tx(&sm.full[q], pair ? 2 * bytes : bytes);
                    bulk_load(buf_t + (size_t)q * kRSubBytes, trow + (size_t)q * SUB_ELEMS, bytes, &sm.full[q]);
                    if (pair) bulk_load(buf_d + (size_t)q * kRSubBytes, drow + (size_t)q * SUB_ELEMS, bytes, &sm.full[q]);
                }
            }
            issued = nsub >= 32 ? 0xffffffffu : ((1u << nsub) - 1u);
        } else {
            E* st = reinterpret_cast<E*>(buf_t);
            E* sd = reinterpret_cast<E*>(buf_d);
            for (int i = tid; i < n; i += kRThreads) {
                st[i] = ld_elem(trow + i);
                if (pair) sd[i] = ld_elem(drow + i);
            }
            __syncthreads();
        }
        if (tid == 0) {
            // the cluster's next queue entry: one per position, or one per sequence when ordered
            if (rank == 0 && (!ordered || j == 0)) next_item = atomicAdd(&p.heads[0], 1) + p.n_clusters;
            tok_ok = true;
            if (pair) {
                const int tok = p.x[(size_t)b * K + j];
                tok_ok = tok >= 0 && tok < V;
                if (tok_ok) {
                    lt = load_logit(tbase + (size_t)target_row(b, j, K) * V + tok);
                    ld = load_logit(dbase + (size_t)draft_row(b, j, K) * V + tok);
                }
                U = uniform_accept(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)j);
            }
        }
    };

    bool have = item < n_items;
    if (have) {
        if (ordered) issue_item((int)item, 0);
        else issue_item((int)(item / (K + 1)), (int)(item % (K + 1)));
    }
    // barriers of every CTA are initialised before any peer arrives on them; the first copies
    // (into this CTA's own memory only) are already under way
    cluster_sync_all();
    if (tid == 0) trace_mark(0, 0);
    while (have) {
        // ---- 1. statistics of the slices as the copies land
        if (tid == 0) trace_mark(1, b * (K + 1) + j);
        const float cb = seq_c(p, b);   // log2(e) / temperature of this sequence
        RowAccT<ENT> at;   // ENT: the target slice also yields its sum e t
        RowAcc ad;
        acc_open(at);
        acc_open(ad);
        for (int q = 0; q < nsub; ++q) {
            if (use_tma && !failed) {
                if (!mbar_wait(&sm.full[q], (full_phase >> q) & 1u, &sm.abort_flag)) failed = true;
            }
            if (failed) break;
            stats_sub<E, ENT>(buf_t, q, n, tid, cb, at);
            if (pair) stats_sub<E, false>(buf_d, q, n, tid, cb, ad);
        }
        if (use_tma) full_phase ^= issued;
        if (tid == 0) trace_mark(2, 0);
        // (max, sum) of the warp's share: the maximum first (shuffles only), then one rescale per
        // thread and a sum -- a much shorter dependent chain than merging (m, s) pairs step by step
        const int par = round & 1;
        {
            float wv = 0.f;
            const float2 pt2 = acc_close(at, cb, &wv), pd2 = acc_close(ad, cb);
            float Mt = pt2.x, Md = pd2.x;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                Mt = fmaxf(Mt, __shfl_xor_sync(0xffffffffu, Mt, off));
                Md = fmaxf(Md, __shfl_xor_sync(0xffffffffu, Md, off));
            }
            const float2 sw = ENT ? rebase_sum_w(pt2.x, pt2.y, wv, Mt, cb) : make_float2(rebase_sum(pt2.x, pt2.y, Mt, cb), 0.f);
            float St = sw.x, Wt = sw.y, Sd = rebase_sum(pd2.x, pd2.y, Md, cb);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                St += __shfl_xor_sync(0xffffffffu, St, off);
                Sd += __shfl_xor_sync(0xffffffffu, Sd, off);
                if (ENT) Wt += __shfl_xor_sync(0xffffffffu, Wt, off);
            }
            // ---- 2. every warp hands its partial result to every CTA of the cluster (itself included)
            const int nx = __shfl_sync(0xffffffffu, next_item, 0);
            if (lane < C) {
                peer_store(map_to_peer(smem_u32(&sm.xstat[par][rank * kRWarps + warp]), (uint32_t)lane),
                           make_float4(Mt, St, Md, Sd));
                if (ENT) peer_store(map_to_peer(smem_u32(&sm.xw[par][rank * kRWarps + warp]), (uint32_t)lane), Wt);
                if (rank == 0 && warp == 0) peer_store(map_to_peer(smem_u32(&sm.xnext[par]), (uint32_t)lane), nx);
                peer_arrive(map_to_peer(smem_u32(&sm.xbar[par]), (uint32_t)lane));
            }
        }
        bool ok = !failed && mbar_wait_cluster(&sm.xbar[par], (uint32_t)(round >> 1) & 1u, &sm.abort_flag);
        ++round;
        if (tid == 0) trace_mark(3, 0);
        // ---- 3. the rows' (max, Z) and the decision
        if (ok && warp == 0) {
            float mt, zt, md, zd, wt;
            merge_exchanged<ENT>(sm.xstat[par], sm.xw[par], C * kRWarps, cb, lane, mt, zt, md, zd, wt);
            if (lane == 0) {
                const double Tb = seq_temperature(p, b), betab = seq_beta(p, b);
                int dec = 1;
                if (!rowstat_ok(mt, zt) || (pair && (!rowstat_ok(md, zd) || !tok_ok)) || !seq_params_ok(Tb, betab)) dec = -1;
                sm.rs_t = make_float2(mt, zt);
                sm.rs_d = pair ? make_float2(md, zd) : make_float2(0.f, 1.f);
                if (pair && dec >= 0) dec = cluster_decide<ENT>(p, b, j, lt, ld, U, sm.rs_t, sm.rs_d, wt, cb, Tb, betab, rank == 0);
                sm.dec = dec;
            }
        }
        if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
        const int dec = sm.dec;
        const long long nxt = sm.xnext[par];
        if (tid == 0) trace_mark(4, dec);
        // ---- 4. the token of a rejected position / the bonus token, from the resident slices
        int writer = (b + j) % C, token = -1;   // reports are spread over the CTAs of the cluster
        double mass = 0.0;
        if (dec >= 0 && (!pair || dec == 0)) {
            const RowNorm rn = make_rownorm(sm.rs_t, sm.rs_d);
            const int nseg = (n + kSegElems - 1) / kSegElems;
            bool resid = pair;
            for (;;) {
                if (resid) slice_segments<E, true>(buf_t, buf_d, n, warp, lane, rn, cb, sm.segsum);
                else slice_segments<E, false>(buf_t, buf_t, n, warp, lane, rn, cb, sm.segsum);
                __syncthreads();
                const int mpar = mround & 1;
                // warp 0: lanes own contiguous runs of segment sums
                const int per = (nseg + 31) / 32;
                const int g0 = min(nseg, lane * per), g1 = min(nseg, g0 + per);
                double loc = 0.0, inc = 0.0;
                if (warp == 0) {
                    for (int g = g0; g < g1; ++g) loc += sm.segsum[g];
                    inc = warp_inclusive_scan(loc, lane);
                    const double total = __shfl_sync(0xffffffffu, inc, 31);
                    if (lane < C) {
                        peer_store(map_to_peer(smem_u32(&sm.xmass[mpar][rank]), (uint32_t)lane), total);
                        peer_arrive(map_to_peer(smem_u32(&sm.mbar2[mpar]), (uint32_t)lane));
                    }
                }
                ok = mbar_wait_cluster(&sm.mbar2[mpar], (uint32_t)(mround >> 1) & 1u, &sm.abort_flag);
                ++mround;
                if (ok && tid == 0) {
                    const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)K);
                    double S = 0.0;
                    for (int i = 0; i < C; ++i) S += sm.xmass[mpar][i];
                    const double target = u * S;
                    double cum = 0.0, before = 0.0, before_last = 0.0;
                    int pick = -1, last = -1;
                    for (int i = 0; i < C && pick < 0; ++i) {
                        const double m_i = sm.xmass[mpar][i];
                        if (m_i > 0.0) {
                            last = i;
                            before_last = cum;
                            if (target < cum + m_i) { pick = i; before = cum; }
                        }
                        cum += m_i;
                    }
                    if (pick < 0) { pick = last; before = before_last; }
                    sm.pick_rank = pick;
                    sm.pick_tin = target - before;
                    sm.pick_S = S;
                }
                if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
                // a rejection implies residual mass; if rounding erased it, draw from P_t instead
                if (resid && !(sm.pick_S * rn.izt >= kTinyMass)) { resid = false; __syncthreads(); continue; }
                break;
            }
            if (failed) break;
            if (sm.pick_rank >= 0) writer = sm.pick_rank;
            mass = sm.pick_S * rn.izt;
            if (rank == sm.pick_rank && warp == 0) {
                const double tin = sm.pick_tin;
                const int per = (nseg + 31) / 32;
                const int g0 = min(nseg, lane * per), g1 = min(nseg, g0 + per);
                double loc = 0.0;
                for (int g = g0; g < g1; ++g) loc += sm.segsum[g];
                const double inc = warp_inclusive_scan(loc, lane);
                const unsigned hit = __ballot_sync(0xffffffffu, tin < inc && loc > 0.0);
                const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
                if (pos) {
                    const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
                    int seg = -1, lastseg = -1;
                    double before = 0.0, before_last = 0.0;
                    if (lane == L) {
                        double run = inc - loc;
                        for (int g = g0; g < g1 && seg < 0; ++g) {
                            const double v = sm.segsum[g];
                            if (v > 0.0) {
                                lastseg = g;
                                before_last = run;
                                if (tin < run + v) { seg = g; before = run; }
                            }
                            run += v;
                        }
                        if (seg < 0) { seg = lastseg; before = before_last; }
                    }
                    seg = __shfl_sync(0xffffffffu, seg, L);
                    before = __shfl_sync(0xffffffffu, before, L);
                    if (seg >= 0) {
                        const int idx = pick_in_segment<E>(buf_t, resid ? buf_d : buf_t, resid, rn, cb, seg * kSegElems,
                                                           min(kSegElems, n - seg * kSegElems), tin - before, lane);
                        token = idx >= 0 ? e0 + idx : -1;
                    }
                }
            }
        }
        // ---- 5. the slices and segment sums are free: start the next item's copies, then let one
        //         CTA report this item and count it; the sequence's last item finishes the sequence
        __syncthreads();
        if (tid == 0) trace_mark(5, token);
        const int rb = b, rj = j;
        if (ordered && dec > 0 && pair) {
            issue_item(b, j + 1);          // accepted: on to the next position (or the extra row) of this sequence
        } else {
            have = nxt < n_items;           // (ordered: the sequence ended here, by rejection, bonus token or bad data)
            if (have) {
                if (ordered) issue_item((int)nxt, 0);
                else issue_item((int)(nxt / (K + 1)), (int)(nxt % (K + 1)));
            }
        }
        if (ordered) {
            // every position a cluster reaches while walking a sequence in order is one the sequence decided
            if (rank == 0 && tid == 0 && rj < K && dec >= 0)
                atomicAdd(&p.heads[dec == 1 ? kCountDirect : (dec == 2 ? kCountPardon : kCountReject)], 1);
            // the cluster owns the whole sequence: one CTA writes its outputs when it ends
            if (rank == writer && warp == 0 && (dec < 0 || rj == K || dec == 0)) {
                int32_t* ot = p.out_tok + (size_t)rb * (K + 1);
                if (dec < 0) {
                    for (int q = lane; q <= K; q += 32) ot[q] = -1;
                    if (lane == 0) {
                        p.out_len[rb] = -1;
                        atomicOr(&p.heads[2], kDevInvalidInput);
                        atomicAdd(&p.heads[kCountInvalid], 1);
                    }
                } else {
                    for (int q = lane; q <= K; q += 32) ot[q] = q < rj ? p.x[(size_t)rb * K + q] : (q == rj ? token : -1);
                    if (lane == 0) {
                        p.out_len[rb] = rj;
                        p.resid[rb] = mass;
                    }
                }
            }
        } else if (rank == writer && warp == 0) {
            int last = 0;
            if (lane == 0) {
                const size_t s = (size_t)rb * (K + 1) + rj;
                p.flag[s] = (signed char)dec;
                p.cand[s] = token;
                p.cand_mass[s] = mass;
                last = ticket_add(&p.ticket[rb]) == K ? 1 : 0;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence();
                finish_sequence(p, rb, lane);
            }
        }
    }

    if (failed || sm.abort_flag) {
        // give copies that may still be in flight a bounded time to land before leaving
        if (use_tma && tid == 0) {
            for (int q = 0; q < kRMaxSub; ++q) {
                if (!((issued >> q) & 1u)) continue;
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(&sm.full[q], ((full_phase ^ issued) >> q) & 1u)) {
                    if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
        if (tid == 0) atomicOr(&p.heads[2], kDevTimeout);
    }
    __syncthreads();
    if (tid == 0) trace_mark(6, 0);
    cluster_sync_all();
}

}  // namespace ears
