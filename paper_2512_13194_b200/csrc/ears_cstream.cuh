// The verification step with thread-block clusters that stream their rows.
//
// Work item = one position of one sequence, as in the resident kernel: the pair (target row k,
// draft row k), or the extra target row K.  A cluster of C CTAs takes an item from a queue; CTA j
// owns the j-th slice of the row(s) and reads it straight from global memory through registers:
//
//   1. softmax statistics (max, sum exp2) of the slices [Sec. 3.1]; for the extra row the sums of
//      2 KB segments are kept in shared memory as well, so that a bonus token needs no second read;
//   2. the partial results and the cluster's next queue entry travel through distributed shared
//      memory (remote stores plus a remote mbarrier arrive per peer);
//   3. every CTA takes the decision of Sec. 3.2 (guards of Sec. 3.3 item 2) from identical numbers;
//   4. the extra row draws its bonus token at once from the segment sums of step 1;
//   5. one CTA reports the item in a per-sequence word of decided / accepted positions.  The report
//      that settles the sequence's first rejection [Sec. 3.1] (every earlier position accepted)
//      publishes a job: the two rows of that one position are read a second time, for the masses
//      max(0, P_t - P_d) and the inverse-CDF pick.  A job is cut into pieces of 16-32 KB per row
//      that the CTAs of the whole launch serve, at most one per round beside their own items and,
//      once their cluster has run out of items, for as long as any sequence is unfinished (one CTA
//      alone is bound by its special-function unit to some 13-19 GB/s on such rows, so a job left
//      to one cluster took 30-40 us).  Whoever reports last (an item or the job) writes the
//      sequence's outputs.
//
// So every logit crosses HBM once for the statistics, and per sequence at most one pair of rows is
// read again (usually from L2).  A rejected position that is not the sequence's first costs nothing.
// A cluster never waits for another cluster while it has items; the only cross-cluster wait is the
// one at the end (CTAs stay to serve pieces until every sequence is finished), which cannot deadlock
// (whoever finishes a sequence waits for nobody) and is time-limited.  Without a shared-memory
// footprint several clusters share an SM and hide each other's exchanges.  What a thread's own
// loads can keep in flight (eight 16-byte loads, 32 KB per CTA) bounds a CTA to some 20 GB/s;
// whenever few CTAs are at work (a batch that does not fill the machine, the end of a launch) that
// bound is the speed of the launch.  Rows of 4-byte logits that are 16-byte aligned therefore pass,
// for their statistics, through a small ring of shared-memory stages filled by bulk asynchronous
// copies (64 KB in flight per CTA, no registers held) and read by all threads of the CTA.
// Ordered mode (EARS_FLAG_STOP_AT_FIRST_REJECT): the queue holds sequences, a cluster walks one
// position by position and stops at its first rejection, whose masses it takes at once (each CTA
// over its slice, without the queue); rows after it are never read.
#pragma once
#include "ears_common.cuh"
#include "ears_math.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"
#include "ears_kernel.cuh"     // pick_in_range
#include "ears_direct.cuh"     // stream_piece, stream_bonus_piece, stream_job_piece
#include "ears_resident.cuh"   // RParams, cluster primitives

namespace ears {

constexpr int kCWarps = kDWarps;          // the streaming helpers stride over this many warps
constexpr int kCThreads = kCWarps * 32;
constexpr int kCSliceAlign = 1024;        // slices are whole 2 KB segments of 2-byte entries (and of 4-byte ones)
constexpr int kCBonusPad = 8;             // stream_bonus_piece may clear up to this many entries past the last segment
#ifndef EARS_C_CTAS
#define EARS_C_CTAS 3
#endif
constexpr int kCCtasPerSm = EARS_C_CTAS;
constexpr int kCFetcher = 32;             // the thread that fetches the next item's token and logits (lane 0 of warp 1)
constexpr int kCStages = 4;               // stages of the CTA's copy ring
constexpr int kCStageBytes = 16384;       // per stage: 16 KB of one row, or 8 KB of each of two rows

struct CSmem {
    alignas(8) uint64_t full[kCStages];   // copy ring: bytes of a stage have landed
    uint64_t xbar[2];                     // statistics exchange, alternating by round
    uint64_t mbar2[2];                    // mass-total exchange, alternating by mass round
    alignas(16) float4 xstat[2][kRMaxCluster * kCWarps];   // (m_t, s_t, m_d, s_d) of every warp of every peer
    float xw[2][kRMaxCluster * kCWarps];  // sum e t of the target slice of every warp of every peer (entropy kernels)
    double xmass[2][kRMaxCluster];        // mass totals of every peer
    int xnext[2];                         // next queue entry of the cluster (written by rank 0)
    int job_b, job_n, job_piece;          // second-pass piece this CTA serves next (job_b < 0: none)
    int my_ticket;                        // ticket of the shared queue this CTA holds (-1: none)
    float tk_lt, tk_ld;                   // the item's token logits and uniform, fetched a round ahead by thread kCFetcher
    double tk_U;
    int tk_ok;
    int drain_state;                      // end of the launch: 0 go on, 1 every sequence is finished, -1 give up
    float2 rs_t, rs_d;                    // (max, Z) of the item's rows
    int dec;                              // 1 accept / row usable, 0 reject, -1 invalid
    int pick_rank;                        // CTA that holds u*S (-1: no mass anywhere)
    double pick_tin, pick_S;
    int abort_flag;
};

// ---- the copy ring ----------------------------------------------------------------------
// All threads of the CTA sweep entries [e0, e0 + n) of one row (r1 = nullptr: 16 KB per stage) or of
// two rows side by side (8 KB of each per stage).  Thread 0 keeps kCStages bulk copies in flight;
// every thread waits for a stage, `process(first half, second half, entries before this stage,
// entries per row in it)` reads it, and after a block-wide barrier the stage is filled again.
// q: stage fills so far (the same in every thread).  -> false if a wait gave up.
// Rows must be 16-byte aligned, e0 and n whole 16-byte vectors.
template <typename E, class F>
__device__ __forceinline__ bool staged_sweep(CSmem& sm, unsigned char* ring, uint32_t& q, const E* r0, const E* r1, int e0, int n,
                                             F process) {
    const int ce = (r1 ? kCStageBytes / 2 : kCStageBytes) / (int)sizeof(E);   // entries per row and stage
    const int nchunks = (n + ce - 1) / ce;
    auto issue = [&](int c) {   // thread 0
        const int stage = (int)((q + (uint32_t)c) % kCStages);
        const uint32_t bytes = (uint32_t)min(ce, n - c * ce) * (uint32_t)sizeof(E);
        unsigned char* dst = ring + (size_t)stage * kCStageBytes;
        mbar_arrive_expect_tx(&sm.full[stage], r1 ? 2 * bytes : bytes);
        bulk_load(dst, r0 + e0 + (size_t)c * ce, bytes, &sm.full[stage]);
        if (r1) bulk_load(dst + kCStageBytes / 2, r1 + e0 + (size_t)c * ce, bytes, &sm.full[stage]);
    };
    if (threadIdx.x == 0)
        for (int c = 0; c < nchunks && c < kCStages; ++c) issue(c);
    bool ok = true;
    for (int c = 0; c < nchunks; ++c) {
        const uint32_t qq = q + (uint32_t)c;
        const int stage = (int)(qq % kCStages);
        if (ok && !mbar_wait(&sm.full[stage], (qq / kCStages) & 1u, &sm.abort_flag)) ok = false;
        const unsigned char* src = ring + (size_t)stage * kCStageBytes;
        if (ok) process(src, src + kCStageBytes / 2, c * ce, min(ce, n - c * ce));
        // everyone is through with the stage (or has given up: then the copies that are still in flight
        // are waited for below, and nothing more is issued)
        if (__syncthreads_or(ok ? 0 : 1)) { ok = false; }
        if (ok && threadIdx.x == 0 && c + kCStages < nchunks) issue(c + kCStages);
        if (!ok) {
            // bounded wait for what was issued beyond this stage, so that no copy lands in memory the CTA has left
            if (threadIdx.x == 0) {
                for (int cc = c + 1; cc < nchunks && cc < c + kCStages; ++cc) {
                    const uint32_t q2 = q + (uint32_t)cc;
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(&sm.full[q2 % kCStages], (q2 / kCStages) & 1u)) {
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                    }
                }
            }
            break;
        }
    }
    q += (uint32_t)nchunks;
    return ok;
}

// A segment sum of the extra row, taken relative to mu, brought to the row's own maximum (mc = m c,
// exact in fp64).  Out of line: the fp64 exp2 would otherwise weigh on the registers of every loop around it.
__device__ __noinline__ double bonus_sum_at_row_maximum(double sum, float mu, double mc) {
    return sum > 0.0 ? sum * exp2((double)mu - mc) : 0.0;
}

// Cluster-wide inverse-CDF pick.  Every CTA holds `nseg` non-negative sums val(g) (fp64) over
// consecutive segments of `seg_elems` entries of its slice, CTAs in slice order.  Totals are
// exchanged through distributed shared memory; every CTA locates the CTA that holds u * S, that CTA
// locates the segment and reads its entries again for the token.  All threads of all CTAs call it.
// -> false if a wait gave up.  token: valid in warp 0 of the CTA sm.pick_rank (-1 elsewhere).
template <typename E, typename ValFn>
__device__ __forceinline__ bool cluster_pick(CSmem& sm, const RParams& p, ValFn val, int nseg, int seg_elems, int b, bool resid,
                                             const E* trow, const E* drow, const RowNorm& rn, float cb, int e0, int n,
                                             int rank, int C, int& mround, int& token) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int mpar = mround & 1;
    const int per = (nseg + 31) / 32;
    const int g0 = min(nseg, lane * per), g1 = min(nseg, g0 + per);
    double loc = 0.0, inc = 0.0;
    token = -1;
    if (warp == 0) {
        for (int g = g0; g < g1; ++g) loc += val(g);
        inc = warp_inclusive_scan(loc, lane);
        const double total = __shfl_sync(0xffffffffu, inc, 31);
        if (lane < C) {
            peer_store(map_to_peer(smem_u32(&sm.xmass[mpar][rank]), (uint32_t)lane), total);
            peer_arrive(map_to_peer(smem_u32(&sm.mbar2[mpar]), (uint32_t)lane));
        }
    }
    const bool ok = mbar_wait_cluster(&sm.mbar2[mpar], (uint32_t)(mround >> 1) & 1u, &sm.abort_flag);
    ++mround;
    if (ok && tid == 0) {
        const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)p.K);
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
    if (__syncthreads_or(ok ? 0 : 1)) return false;
    // a rejection implies residual mass; if rounding erased it the caller draws from P_t instead
    if (resid && !(sm.pick_S * rn.izt >= kTinyMass)) return true;
    if (rank == sm.pick_rank && warp == 0) {
        const double tin = sm.pick_tin;
        const unsigned hit = __ballot_sync(0xffffffffu, tin < inc && loc > 0.0);
        const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
        if (pos) {
            const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
            int seg = -1, lastseg = -1;
            double before = 0.0, before_last = 0.0;
            if (lane == L) {
                double run = inc - loc;
                for (int g = g0; g < g1 && seg < 0; ++g) {
                    const double v = val(g);
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
            if (seg >= 0)
                token = pick_in_range<E>(trow, drow, resid, rn, cb, e0 + seg * seg_elems, min(seg_elems, n - seg * seg_elems),
                                         tin - before, p.V, lane);
        }
    }
    return true;
}

// First rejection that a word of decided (low 32 bits) and accepted (high 32 bits) positions settles:
// the lowest rejected position, provided every position before it has been decided (then they were
// all accepted); -1 while that is open or when nothing decided so far was rejected.
__device__ __forceinline__ int settled_first_rejection(unsigned long long m, int K) {
    const uint32_t decided = (uint32_t)m, accepted = (uint32_t)(m >> 32);
    const uint32_t rej = decided & ~accepted & ((1u << K) - 1u);
    if (!rej) return -1;
    const int n = __ffs(rej) - 1;
    const uint32_t below = (1u << n) - 1u;
    return (decided & below) == below ? n : -1;
}

// The word of a sequence: bit k of the low half = position k (K = the extra row) has reported, bit k of
// the high half = it was not rejected; the top bit = the second-pass job has reported.  The sequence is
// complete with the report that makes "all K+1 positions in, and the job too if a position was
// rejected" true; reports only add bits, so exactly one report sees it (none follows it).
constexpr unsigned long long kJobReported = 1ull << 63;
__device__ __forceinline__ bool sequence_complete(unsigned long long m, int K) {
    const uint32_t decided = (uint32_t)m, accepted = (uint32_t)(m >> 32);
    const uint32_t items = (2u << K) - 1u;   // K <= 30
    if ((decided & items) != items) return false;
    const bool rejected = (decided & ~accepted & ((1u << K) - 1u)) != 0;
    return !rejected || (m & kJobReported) != 0;
}
// Adds bits to that word with release + acquire semantics at device scope in the atomic itself: the
// reporter's stores are visible to whoever sees the bits, and earlier reporters' stores to the reporter.
__device__ __forceinline__ unsigned long long seqmask_or(unsigned long long* addr, unsigned long long bits) {
    unsigned long long old;
    asm volatile("atom.or.acq_rel.gpu.b64 %0, [%1], %2;" : "=l"(old) : "l"(addr), "l"(bits) : "memory");
    return old;
}

// Called by one warp once everything of sequence b is in: first rejection [Sec. 3.1], the accepted
// prefix and the token drawn at that position (or the bonus token).  With job_pending the slot of a
// rejected position is left to the second-pass job that is yet to run (K > 30 only).
// -> n in [0, K], or -1 for an invalid sequence.
__device__ __forceinline__ int finish_streamed_sequence(const RParams& p, int b, int lane, bool job_pending) {
    const int K = p.K;
    const signed char* fl = p.flag + (size_t)b * (K + 1);
    int32_t* ot = p.out_tok + (size_t)b * (K + 1);
    if (K < 32) {
        // one lane per position: everything the outputs need is asked for at once (this runs at the very
        // end of a launch, where every dependent round trip shows)
        int f = 1, xk = -1, ck = -1;
        double cm = 0.0;
        if (lane <= K) {
            f = *reinterpret_cast<const volatile signed char*>(fl + lane);
            ck = __ldcg(p.cand + (size_t)b * (K + 1) + lane);
            cm = __ldcg(p.cand_mass + (size_t)b * (K + 1) + lane);
            if (lane < K) xk = p.x[(size_t)b * K + lane];
        }
        const unsigned rej = __ballot_sync(0xffffffffu, lane < K && f == 0);
        const bool bad = __any_sync(0xffffffffu, f < 0);
        if (bad) {
            if (lane <= K) ot[lane] = -1;
            if (lane == 0) {
                p.out_len[b] = -1;
                atomicOr(&p.heads[2], kDevInvalidInput);
                atomicAdd(&p.heads[kCountInvalid], 1);
            }
            return -1;
        }
        const int n = rej ? __ffs(rej) - 1 : K;
        count_decisions(p.heads, min(n + 1, K), lane, [f](int) { return f; });
        const bool mine = n == K || !job_pending;   // the slot n is filled here
        if (lane < n) ot[lane] = xk;
        else if (lane > n && lane <= K) ot[lane] = -1;
        else if (lane == n && mine) { ot[lane] = ck; p.resid[b] = cm; }
        if (lane == 0) p.out_len[b] = n;
        return n;
    }
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
    if (bad) {
        for (int q = lane; q <= K; q += 32) ot[q] = -1;
        if (lane == 0) {
            p.out_len[b] = -1;
            atomicOr(&p.heads[2], kDevInvalidInput);
            atomicAdd(&p.heads[kCountInvalid], 1);
        }
        return -1;
    }
    const int n = first_reject;
    count_decisions(p.heads, min(n + 1, K), lane, [fl](int k) { return (int)*reinterpret_cast<const volatile signed char*>(fl + k); });
    const bool mine = n == K || !job_pending;   // the slot n is filled here
    for (int q = lane; q <= K; q += 32) {
        if (q < n) ot[q] = p.x[(size_t)b * K + q];
        else if (q > n) ot[q] = -1;
        else if (mine) ot[q] = __ldcg(p.cand + (size_t)b * (K + 1) + n);
    }
    if (lane == 0) {
        p.out_len[b] = n;
        if (mine) p.resid[b] = __ldcg(p.cand_mass + (size_t)b * (K + 1) + n);
    }
    return n;
}

// ---- second-pass jobs, shared by all CTAs of the launch --------------------------------
// A job = (sequence b, its first rejected position n); its rows' statistics are in p.rowstat before
// it is published.  Published jobs form a queue (p.ready, filled in the order of p.heads[3]); a job
// has p.parts2 pieces of p.job_elems entries.  Pieces are handed out by one counter for the whole
// queue (p.heads[4]): ticket i stands for piece i % parts2 of the job in slot i / parts2, whether or
// not that job has been published yet.  A CTA with nothing else to do takes a ticket and waits for
// its slot: when a job appears, the parts2 CTAs that hold its tickets serve it at once, with no
// contention and one atomic per piece.  A CTA that still has items takes a ticket only while the
// counter is behind the publications, i.e. when a piece is there to be served right away.
// p.ticket2[b] counts the pieces of b's job that are done; the CTA that completes the last one
// draws the token.

// One thread publishes a job (its rowstat entry and whatever else a server reads were written
// before by this thread, or are ordered before by a fence of the caller).
__device__ __forceinline__ void publish_job(const RParams& p, int b, int n) {
    __threadfence();
    const int slot = atomicAdd(&p.heads[3], 1);
    *reinterpret_cast<volatile unsigned long long*>(&p.ready[slot]) = ((unsigned long long)(b + 1) << 32) | (unsigned)n;
}

// A sequence is finished (its outputs are complete): lets the CTAs that stay to serve pieces leave.
__device__ __forceinline__ void count_finished(const RParams& p) {
    __threadfence();
    atomicAdd(&p.heads[1], 1);
}

// What lane 0 of warp 0 reads of the queue at the start of a round, so that it costs no wait later:
// jobs published, tickets given out, and the entry of the slot of the ticket this CTA holds.
struct JobPoll { int published, given; unsigned long long e; };

__device__ __forceinline__ unsigned long long ticket_slot_entry(const RParams& p, int ticket) {
    const int slot = ticket / p.parts2;
    return slot < p.B ? *reinterpret_cast<const volatile unsigned long long*>(&p.ready[slot]) : 0ull;
}

__device__ __forceinline__ JobPoll poll_jobs(const RParams& p, const CSmem& sm) {
    JobPoll q;
    q.published = *reinterpret_cast<const volatile int*>(&p.heads[3]);
    q.given = *reinterpret_cast<const volatile int*>(&p.heads[4]);
    q.e = sm.my_ticket >= 0 ? ticket_slot_entry(p, sm.my_ticket) : 0ull;
    return q;
}

// Thread 0 decides which second-pass piece the CTA serves next and leaves it in shared memory
// (job_b < 0: none): the piece of the ticket it holds, once that piece's job is published.
// turn < 0: the CTA has no items left, so it takes a ticket whatever the state of the queue.  Otherwise (turn = its round) it takes one only if the
// polled counters say pieces are waiting, and only if it is among as many CTAs as there are such
// pieces (a window of CTA indices that moves with the round): the CTAs of a launch poll at about
// the same time and see the same counters, and if all of them took a ticket most would end up
// holding one for a job that is yet to come, which then has to wait for a busy CTA.
__device__ __forceinline__ void claim_job(const RParams& p, CSmem& sm, const JobPoll& q, int turn) {
    const int P2 = p.parts2;
    int jb = -1, jn = 0, piece = 0;
    {
        unsigned long long e = q.e;
        const int waiting = q.published * P2 - q.given;
        const bool idle = turn < 0;
        if (sm.my_ticket < 0 && (idle || (int)((blockIdx.x + (unsigned)turn * 37u) % gridDim.x) < waiting)) {
            sm.my_ticket = atomicAdd(&p.heads[4], 1);
            e = ticket_slot_entry(p, sm.my_ticket);
        }
        if (sm.my_ticket >= 0 && e != 0) {
            jb = (int)(e >> 32) - 1;
            jn = (int)(unsigned)e;
            piece = sm.my_ticket % P2;
            sm.my_ticket = -1;
        }
    }
    sm.job_b = jb; sm.job_n = jn; sm.job_piece = piece;
}

// The CTA that completed a job's last piece draws the token from the stored segment sums (one warp):
// token = smallest j with u S < C_j over max(0, P_t - P_d) of position n [Sec. 3.1; speculative
// sampling's residual draw], from P_t if rounding left the residual without mass.
template <typename E>
__device__ __forceinline__ int select_job_token(const RParams& p, int b, int n, int lane, double* mass_out) {
    const int K = p.K, V = p.V;
    const float cj = seq_c(p, b);
    const E* trow = reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, n, K) * V;
    const E* drow = reinterpret_cast<const E*>(p.d) + (size_t)draft_row(b, n, K) * V;
    const float4 rs = __ldcg(&p.rowstat[(size_t)b * (K + 1) + n]);
    const RowNorm rn = make_rownorm(make_float2(rs.x, rs.y), make_float2(rs.z, rs.w));
    const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)K);
    const double* ss = p.segsums + (size_t)b * p.nseg;
    double S = 0.0, before = 0.0;
    const int seg = pick_block([ss](int g) { return __ldcg(ss + g); }, p.nseg, u, lane, &S, &before);
    int tok;
    double S_used = S;
    if (seg < 0 || !(S * rn.izt >= kTinyMass)) tok = warp_sample_pt_slow<E>(trow, V, rn, cj, u, lane, &S_used);
    else tok = pick_in_range<E>(trow, drow, true, rn, cj, seg * kSegElems, kSegElems, u * S - before, V, lane);
    *mass_out = S_used * rn.izt;
    return tok;
}

// All threads of the CTA: the piece that thread 0 left in shared memory (claim_job, then a block-wide
// barrier).  -> false if there was none.
template <typename E>
__device__ __forceinline__ bool serve_claimed_piece(const RParams& p, CSmem& sm, bool vec, bool early) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int jb = sm.job_b, jn = sm.job_n, piece = sm.job_piece;
    if (jb < 0) return false;
    const int K = p.K, V = p.V;
    __threadfence();   // the publication was seen: what preceded it (the rows' statistics) is visible
    const float cj = seq_c(p, jb);
    const E* jt = reinterpret_cast<const E*>(p.t) + (size_t)target_row(jb, jn, K) * V;
    const E* jd = reinterpret_cast<const E*>(p.d) + (size_t)draft_row(jb, jn, K) * V;
    const float4 rs = __ldcg(&p.rowstat[(size_t)jb * (K + 1) + jn]);
    const RowNorm rn = make_rownorm(make_float2(rs.x, rs.y), make_float2(rs.z, rs.w));
    const int e0 = min(V, piece * p.job_elems), e1 = min(V, e0 + p.job_elems);
    stream_job_piece<E, true>(jt, jd, e0, e1, vec, rn, cj, warp, lane, p.segsums + (size_t)jb * p.nseg);
    __threadfence();   // the sums are visible before the piece counts as done
    __syncthreads();
    if (warp == 0) {
        int last = 0;
        if (lane == 0) last = ticket_add(&p.ticket2[jb]) == p.parts2 - 1 ? 1 : 0;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            __threadfence();
            double mass = 0.0;
            const int jtoken = select_job_token<E>(p, jb, jn, lane, &mass);
            if (early) {
                // the job reports like an item; if it is the last of the sequence to do so it finishes it
                int fin = 0;
                if (lane == 0) {
                    const size_t s = (size_t)jb * (K + 1) + jn;
                    p.cand[s] = jtoken;
                    p.cand_mass[s] = mass;
                    fin = sequence_complete(seqmask_or(p.seqmask + jb, kJobReported) | kJobReported, K) ? 1 : 0;
                }
                fin = __shfl_sync(0xffffffffu, fin, 0);
                if (fin) {
                    __threadfence();
                    finish_streamed_sequence(p, jb, lane, false);
                    if (lane == 0) count_finished(p);
                }
            } else if (lane == 0) {
                // the rest of the sequence's outputs were written by whoever published the job
                p.out_tok[(size_t)jb * (K + 1) + jn] = jtoken;
                p.resid[jb] = mass;
                count_finished(p);
            }
            if (lane == 0) trace_mark(7, jtoken);
        }
    }
    return true;
}

template <typename E, bool ENT>
__global__ void __launch_bounds__(kCThreads, kCCtasPerSm) ears_cstream_kernel(const RParams p) {
    extern __shared__ unsigned char smem_raw[];
    CSmem& sm = *reinterpret_cast<CSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    unsigned char* area = reinterpret_cast<unsigned char*>(&sm) + ((sizeof(CSmem) + 127) & ~size_t(127));
    BonusSeg* const bseg = reinterpret_cast<BonusSeg*>(area);   // the extra row's sums per 2 KB
    unsigned char* const ring = area + p.buf_bytes;             // the copy ring (behind the sums; 128-byte aligned)
    uint32_t ring_q = 0;                                        // stage fills so far
    constexpr int BSEG = kBonusSegBytes / (int)sizeof(E);       // entries per bonus segment
    const int K = p.K, V = p.V, C = p.C;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / C;
    const bool ordered = p.ordered != 0;
    // first rejections are settled as the reports come in when the decided / accepted bits of a sequence fit one word
    const bool early = !ordered && K <= 30;
    const long long n_items = ordered ? (long long)p.B : (long long)p.B * (K + 1);
    const bool vec = p.use_tma != 0;   // rows are 16-byte aligned: 16-byte loads
    const E* tbase = reinterpret_cast<const E*>(p.t);
    const E* dbase = reinterpret_cast<const E*>(p.d);

    if (tid == 0) trace_mark(0, 0);
    clear_next_counters(p);
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&sm.xbar[i], (unsigned)(C * kCWarps)); mbar_init(&sm.mbar2[i], (unsigned)C); }
        for (int i = 0; i < kCStages; ++i) mbar_init(&sm.full[i], 1u);
        sm.abort_flag = 0;
        sm.job_b = -1;
        sm.my_ticket = -1;
        sm.drain_state = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const int e0 = rank * p.slice;                         // this CTA's slice of every row
    const int n = max(0, min(p.slice, V - e0));
    int round = 0, mround = 0;                             // exchanges so far (the same in every CTA of the cluster)
    bool failed = false;
    int b = 0, j = 0;
    // what thread kCFetcher fetches ahead for an item's decision: the token's two logits and the uniform
    float lt = 0.f, ld = 0.f, nx_lt = 0.f, nx_ld = 0.f;
    double U = 0.0, nx_U = 0.0;
    bool tok_ok = true, nx_tok_ok = true;
    int next_item = 0;

    auto fetch_token = [&](int fb, int fj) {   // thread kCFetcher
        nx_tok_ok = true;
        if (fj < K) {
            const int tok = p.x[(size_t)fb * K + fj];
            nx_tok_ok = tok >= 0 && tok < V;
            if (nx_tok_ok) {
                nx_lt = load_logit(tbase + (size_t)target_row(fb, fj, K) * V + tok);
                nx_ld = load_logit(dbase + (size_t)draft_row(fb, fj, K) * V + tok);
            }
            nx_U = uniform_accept(p.seed, p.offset, (uint32_t)(p.b_first + fb), (uint32_t)fj);
        }
    };
    auto take_item = [&](int nb, int nj) {
        b = nb;
        j = nj;
        if (tid == 0) {
            // the cluster's next queue entry: one per position, or one per sequence when ordered
            if (rank == 0 && (!ordered || j == 0)) next_item = atomicAdd(&p.heads[0], 1) + p.n_clusters;
        }
    };

    bool have = cluster_id < n_items;
    if (have) {
        const int fb = ordered ? cluster_id : cluster_id / (K + 1), fj = ordered ? 0 : cluster_id % (K + 1);
        if (tid == kCFetcher) fetch_token(fb, fj);
        take_item(fb, fj);
    }
    // barriers of every CTA are initialised before any peer arrives on them
    cluster_sync_all();

    while (have) {
        const bool pair = j < K;
        const float cb = seq_c(p, b);    // log2(e) / temperature of this sequence
        const E* const trow = tbase + (size_t)target_row(b, j, K) * V;
        const E* const drow = dbase + (size_t)draft_row(b, pair ? j : 0, K) * V;
        // a look at the queue of second-pass jobs, taken now so that it costs no wait after the sweep
        JobPoll polled{0, 0, 0ull};
        if (tid == 0) polled = poll_jobs(p, sm);
        // ---- 1. statistics of this CTA's slices
        if (tid == 0) trace_mark(1, b * (K + 1) + j);
        float2 pt2 = make_float2(-INFINITY, 0.f), pd2 = make_float2(-INFINITY, 0.f);
        float wv = 0.f;   // ENT: the thread's sum e t over the target slice
        // 4-byte logits take the copy ring (measured on B200, 64 sequences of 1 MB rows: 121 us against 184);
        // 2-byte logits do twice the arithmetic per staged byte and lose to their own loads there
        // (32 sequences of 256 KB rows: 55 us against 47), so they keep the register path
        const bool staged = vec && sizeof(E) == 4;
        if (staged && pair) {
            // through the copy ring: 8 KB of each row per stage, two vectors of each per thread
            constexpr int N = Words<E>::N;
            RowAccT<ENT> at;
            RowAcc ad;
            acc_open(at);
            acc_open(ad);
            const bool swept = staged_sweep<E>(sm, ring, ring_q, trow, drow, e0, n,
                [&](const unsigned char* bt, const unsigned char* bd, int, int cnt) {
                    const int nv = cnt / N;   // whole vectors: rows and slices are
                    uint4 wt[2], wd[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int v = tid + h * kCThreads;
                        wt[h] = v < nv ? reinterpret_cast<const uint4*>(bt)[v] : Words<E>::minus_inf();
                        wd[h] = v < nv ? reinterpret_cast<const uint4*>(bd)[v] : Words<E>::minus_inf();
                    }
                    fold_vectors<E, 2, ENT>(wt, cb, at);
                    fold_vectors<E, 2, false>(wd, cb, ad);
                });
            if (!swept) { failed = true; break; }
            pt2 = acc_close(at, cb, &wv);
            pd2 = acc_close(ad, cb);
        } else if (staged) {
            // the extra row through the copy ring: 16 KB per stage, warp w takes its 2 KB block w, keeps a
            // warp-uniform running maximum and leaves (sum, reference) of the block behind
            constexpr int N = Words<E>::N, PN = N / 2, VPL = BSEG / N / 32;
            RowAcc a;
            acc_open(a);
            const f32x2 c2 = pack2(cb, cb);
            const bool swept = staged_sweep<E>(sm, ring, ring_q, trow, (const E*)nullptr, e0, n,
                [&](const unsigned char* bt, const unsigned char*, int before, int cnt) {
                    const int first = warp * BSEG;   // this warp's block within the stage
                    if (first >= cnt) return;
                    uint4 w[VPL];
#pragma unroll
                    for (int i = 0; i < VPL; ++i) {
                        const int k0 = first + (i * 32 + lane) * N;
                        w[i] = k0 < cnt ? reinterpret_cast<const uint4*>(bt)[k0 / N] : Words<E>::minus_inf();
                    }
                    float cm = Words<E>::template vmax_all<VPL>(w);
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, off));
                    acc_raise(a, cm, cb);
                    const f32x2 nmu2 = pack2(-a.mu, -a.mu);
                    f32x2 cs[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
                    for (int i = 0; i < VPL; ++i) {
                        f32x2 q2[PN];
                        Words<E>::pairs(w[i], q2);
#pragma unroll
                        for (int u = 0; u < PN; u += 2) {
                            cs[0] = add2(cs[0], ex2_pair(fma2(q2[u], c2, nmu2)));
                            cs[1] = add2(cs[1], ex2_pair(fma2(q2[u + 1], c2, nmu2)));
                        }
                    }
                    a.s[0] = add2(a.s[0], cs[0]);
                    a.s[1] = add2(a.s[1], cs[1]);
                    float q0, q1;
                    unpack2(add2(cs[0], cs[1]), q0, q1);
                    double tot = (double)(q0 + q1);   // a lane's few terms in fp32, lanes in fp64
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, off);
                    if (lane == 0) bseg[(before + first) / BSEG] = BonusSeg{tot, a.mu, 0.f};
                });
            if (!swept) { failed = true; break; }
            pt2 = acc_close(a, cb);
        } else {
            if (pair) {
                pt2 = stream_piece<E, kCThreads, ENT>(trow, e0, e0 + n, vec, cb, tid, &wv);
                pd2 = stream_piece<E, kCThreads>(drow, e0, e0 + n, vec, cb, tid);
            } else {
                pt2 = stream_bonus_piece<E>(trow, e0, e0 + n, vec, cb, warp, lane, bseg - e0 / BSEG);
            }
        }
        if (tid == 0) trace_mark(2, 0);
        // what was fetched ahead for this item goes to shared memory now that the sweep is over (the barrier
        // of the exchange below orders it before the decision)
        if (tid == kCFetcher) { sm.tk_lt = nx_lt; sm.tk_ld = nx_ld; sm.tk_U = nx_U; sm.tk_ok = nx_tok_ok ? 1 : 0; }
        // (max, sum) of the warp's share: the maximum first (shuffles only), then one rescale per thread and a sum
        const int par = round & 1;
        {
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
            // ---- 2. every warp hands its partial result to every CTA of the cluster (itself included);
            //         warp 0 of rank 0 adds the cluster's next queue entry
            const int nx = __shfl_sync(0xffffffffu, next_item, 0);
            if (C == 1) {
                // a cluster of one: plain shared memory and the block-wide barrier below do
                if (lane == 0) {
                    sm.xstat[par][warp] = make_float4(Mt, St, Md, Sd);
                    if (ENT) sm.xw[par][warp] = Wt;
                    if (warp == 0) sm.xnext[par] = nx;
                }
            } else if (lane < C) {
                peer_store(map_to_peer(smem_u32(&sm.xstat[par][rank * kCWarps + warp]), (uint32_t)lane),
                           make_float4(Mt, St, Md, Sd));
                if (ENT) peer_store(map_to_peer(smem_u32(&sm.xw[par][rank * kCWarps + warp]), (uint32_t)lane), Wt);
                if (warp == 0 && rank == 0) peer_store(map_to_peer(smem_u32(&sm.xnext[par]), (uint32_t)lane), nx);
                peer_arrive(map_to_peer(smem_u32(&sm.xbar[par]), (uint32_t)lane));
            }
        }
        bool ok = C == 1 || mbar_wait_cluster(&sm.xbar[par], (uint32_t)(round >> 1) & 1u, &sm.abort_flag);
        ++round;
        if (tid == 0) trace_mark(3, 0);
        if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
        // the cluster's next queue entry, known to every CTA now
        const long long nxt = sm.xnext[par];
        const bool q_have = nxt < n_items;
        const int qb = q_have ? (ordered ? (int)nxt : (int)(nxt / (K + 1))) : 0;
        const int qj = (q_have && !ordered) ? (int)(nxt % (K + 1)) : 0;
        // ---- 3. the rows' (max, Z) and the decision
        if (warp == 0) {
            float mt, zt, md, zd, wt;
            merge_exchanged<ENT>(sm.xstat[par], sm.xw[par], C * kCWarps, cb, lane, mt, zt, md, zd, wt);
            if (lane == 0) {
                // what was fetched ahead for this item is taken over only now: the loads (two dependent
                // misses for the first item of a launch) have had the whole sweep to land
                lt = sm.tk_lt; ld = sm.tk_ld; U = sm.tk_U; tok_ok = sm.tk_ok != 0;
                const double Tb = seq_temperature(p, b), betab = seq_beta(p, b);
                int dec = 1;
                if (!rowstat_ok(mt, zt) || (pair && (!rowstat_ok(md, zd) || !tok_ok)) || !seq_params_ok(Tb, betab)) dec = -1;
                sm.rs_t = make_float2(mt, zt);
                sm.rs_d = pair ? make_float2(md, zd) : make_float2(0.f, 1.f);
                if (pair && dec >= 0) dec = cluster_decide<ENT>(p, b, j, lt, ld, U, sm.rs_t, sm.rs_d, wt, cb, Tb, betab, rank == 0);
                sm.dec = dec;
            }
        }
        __syncthreads();
        const int dec = sm.dec;
        if (tid == 0) trace_mark(4, dec);
        if (tid == kCFetcher) {
            // the next item's token and its two logits, asked for by a thread of a warp that has nothing to do
            // until this item is reported (the address of the logits waits for the token: a round trip that the
            // deciding warp does not have to sit through); the loads land during the next sweep
            // (walking a sequence in order, an accepted position is followed by the next one)
            if (ordered && pair && dec > 0) fetch_token(b, j + 1);
            else if (q_have) fetch_token(qb, qj);
        }
        // ---- 4. the extra row draws its bonus token at once from the segment sums of step 1
        int writer = (b + j) % C, token = -1;   // reports are spread over the CTAs of the cluster
        double mass = 0.0;
        if (!pair && dec >= 0) {
            const RowNorm rn = make_rownorm(sm.rs_t, sm.rs_d);
            const double mc = (double)rn.mt * (double)cb;   // exact: two fp32 factors
            const BonusSeg* bs = bseg;
            // the terms of a segment were exp2(l c - mu): bring its sum to the row's own maximum (fp64: no new error)
            auto val = [bs, mc](int g) { return bonus_sum_at_row_maximum(bs[g].sum, bs[g].mu, mc); };
            if (!cluster_pick<E>(sm, p, val, (n + BSEG - 1) / BSEG, BSEG, b, false, trow, trow, rn, cb, e0, n, rank, C, mround, token)) {
                failed = true;
                break;
            }
            if (sm.pick_rank >= 0) writer = sm.pick_rank;
            mass = sm.pick_S * rn.izt;
        }
        // ---- 5. one CTA reports the item and counts it; the sequence's last item finishes the sequence;
        //         a first rejection is published as a second-pass job
        bool seq_goes_on = false;
        if (ordered) {
            seq_goes_on = dec > 0 && pair;
            // every position a cluster reaches while walking a sequence in order is one the sequence decided
            if (rank == 0 && tid == 0 && pair && dec >= 0)
                atomicAdd(&p.heads[dec == 1 ? kCountDirect : (dec == 2 ? kCountPardon : kCountReject)], 1);
            if (rank == writer && warp == 0 && !seq_goes_on) {
                int32_t* ot = p.out_tok + (size_t)b * (K + 1);
                if (dec < 0) {
                    for (int q = lane; q <= K; q += 32) ot[q] = -1;
                    if (lane == 0) {
                        p.out_len[b] = -1;
                        atomicOr(&p.heads[2], kDevInvalidInput);
                        atomicAdd(&p.heads[kCountInvalid], 1);
                        count_finished(p);
                    }
                } else {
                    for (int q = lane; q <= K; q += 32) {
                        if (q < j) ot[q] = p.x[(size_t)b * K + q];
                        else if (q > j) ot[q] = -1;
                        else if (!pair) ot[q] = token;        // the bonus token; a rejected slot is the job's to fill
                    }
                    if (lane == 0) {
                        p.out_len[b] = j;
                        if (!pair) {
                            p.resid[b] = mass;
                            count_finished(p);
                        }   // (the first rejection of a sequence walked in order: its token is drawn below)
                    }
                }
            }
        } else if (rank == writer && warp == 0) {
            int last = 0;
            if (lane == 0) {
                const size_t s = (size_t)b * (K + 1) + j;
                p.flag[s] = (signed char)dec;
                p.cand[s] = token;
                p.cand_mass[s] = mass;
                p.rowstat[s] = make_float4(sm.rs_t.x, sm.rs_t.y, sm.rs_d.x, sm.rs_d.y);
                if (early) {
                    // decided, and accepted unless rejected (an unusable position counts as accepted here: it
                    // must not ask for masses; the flag array remembers it and invalidates the sequence).
                    // One atomic on the sequence's word does it all: it releases the stores above, tells
                    // whether this report settles the first rejection, and whether it is the sequence's last.
                    const unsigned long long bit = 1ull << j;
                    const unsigned long long add = bit | (dec != 0 ? bit << 32 : 0ull);
                    const unsigned long long old = seqmask_or(p.seqmask + b, add);
                    const int n_now = settled_first_rejection(old | add, K);
                    if (n_now >= 0 && settled_first_rejection(old, K) < 0) publish_job(p, b, n_now);   // settled by this report
                    last = sequence_complete(old | add, K) ? 1 : 0;
                } else {
                    last = ticket_add(&p.ticket[b]) == K ? 1 : 0;
                }
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence();
                const int nfirst = finish_streamed_sequence(p, b, lane, !early);
                if (lane == 0) {
                    if (!early && nfirst >= 0 && nfirst < K) publish_job(p, b, nfirst);   // the job fills slot nfirst
                    else count_finished(p);
                }
            }
        }
        if (tid == 0) trace_mark(5, token);
        if (ordered && dec == 0) {
            // The first rejection of a sequence walked in order: every CTA of the cluster knows it, so the
            // cluster takes the masses of that position at once, without the queue: each CTA over its own
            // slice into shared memory (the area of the extra row's sums is as large and not in use: a
            // rejected position is not followed by that row), then the cluster-wide pick of step 4.
            const RowNorm rn = make_rownorm(sm.rs_t, sm.rs_d);
            double* const segsum = reinterpret_cast<double*>(area);
            double* so = segsum - e0 / kSegElems;    // sums land at index (entry - e0) / kSegElems
            const double* ss = segsum;
            auto val = [ss](int g) { return ss[g]; };
            int jtoken = -1;
            bool resid = true;
            for (;;) {
                if (resid) stream_job_piece<E, true>(trow, drow, e0, e0 + n, vec, rn, cb, warp, lane, so);
                else stream_job_piece<E, false>(trow, trow, e0, e0 + n, vec, rn, cb, warp, lane, so);
                __syncthreads();
                if (!cluster_pick<E>(sm, p, val, (n + kSegElems - 1) / kSegElems, kSegElems, b, resid, trow, drow, rn, cb, e0, n, rank, C,
                                     mround, jtoken)) {
                    failed = true;
                    break;
                }
                // a rejection implies residual mass; if rounding erased it, draw from P_t instead
                if (resid && !(sm.pick_S * rn.izt >= kTinyMass)) { resid = false; __syncthreads(); continue; }
                break;
            }
            if (failed) break;
            if (warp == 0 && lane == 0 && (rank == sm.pick_rank || (sm.pick_rank < 0 && rank == 0))) {
                p.out_tok[(size_t)b * (K + 1) + j] = jtoken;
                p.resid[b] = sm.pick_S * rn.izt;
                count_finished(p);
                trace_mark(7, jtoken);
            }
        }
        // ---- 6. one piece of a published second-pass job, if the look at the start of the round found one waiting
        if (tid == 0) claim_job(p, sm, polled, round);
        __syncthreads();     // the claim is known; shared memory of this round (decision, sums) is free again
        serve_claimed_piece<E>(p, sm, vec, early);
        // ---- on to the next item
        if (seq_goes_on) {
            take_item(b, j + 1);
        } else {
            have = q_have;
            if (have) take_item(qb, qj);
        }
    }
    // ---- the cluster has run out of items: its CTAs stay and serve second-pass pieces until every
    //      sequence of the batch is finished (by whichever CTA).  A sequence is finished by CTAs that
    //      wait for nobody, so this cannot deadlock; it is time-limited like every other wait.
    if (!failed) {
        unsigned long long wait_t0 = 0;
        for (;;) {
            if (tid == 0) {
                const JobPoll q{0, 0, sm.my_ticket >= 0 ? ticket_slot_entry(p, sm.my_ticket) : 0ull};
                claim_job(p, sm, q, -1);
                int st = 0;
                if (sm.job_b < 0) {
                    if (*reinterpret_cast<volatile int*>(&p.heads[1]) >= p.B) {
                        st = 1;
                    } else if (*reinterpret_cast<volatile int*>(&p.heads[2]) & kDevTimeout) {
                        st = -1;   // another CTA gave up: the count will never be reached
                    } else {
                        const unsigned long long now = global_timer_ns();
                        if (wait_t0 == 0) wait_t0 = now;
                        else if (now - wait_t0 > kIdleLimitNs) st = -1;
                        __nanosleep(200);
                    }
                }
                sm.drain_state = st;
            }
            __syncthreads();
            const int st = sm.drain_state;
            const bool served = serve_claimed_piece<E>(p, sm, vec, early);
            __syncthreads();   // everyone has read the claim and the state before warp 0 writes them again
            if (served) continue;
            if (st > 0) break;
            if (st < 0) { failed = true; break; }
        }
    }
    if (tid == 0) trace_mark(6, 0);
    if (failed || sm.abort_flag) {
        if (tid == 0) atomicOr(&p.heads[2], kDevTimeout);
    }
    __syncthreads();
    cluster_sync_all();   // no CTA leaves while a peer may still store into it
}

}  // namespace ears
