// The verification step for long rows, streamed straight from global memory.
//
// Every warp of every CTA computes; there is no shared-memory staging and no loader.  A thread
// keeps eight 16-byte loads in flight, folds them into its running (max, sum exp2) [softmax
// statistics, Sec. 3.1] and moves on, so that warps never march in step from barrier to barrier
// and the special-function pipe is busy evenly (on 2-byte logits this is worth 60 % over a
// ring of staged slots with dedicated loader and consumer warps).  Work is cut into units (a
// piece of one row) pulled from an atomic queue in sequence-major order:
//
//   unit of an ordinary row   all threads stride over the piece; block-wide reduction; thread 0
//                             stores the piece's (m, s) and counts it (per row, per sequence);
//   unit of the extra row K   warps take whole 2 KB segments instead and also leave the sum of
//                             every segment behind, so that a bonus token can be drawn later
//                             without reading the row again;
//   last piece of a sequence  warp 0 of the CTA that delivered it merges the pieces, decides
//                             every position (Sec. 3.2 with the guards of Sec. 3.3 item 2),
//                             finds the first rejection (Sec. 3.1) and either draws the bonus
//                             token at once or publishes the sequence for a second pass;
//   second-pass piece         the two rows of the rejected position are cut into pieces that all
//                             CTAs serve ahead of new units (they were read moments ago and are
//                             mostly still in L2): sums of max(0, P_t - P_d) per 256 entries; the
//                             CTA delivering the last piece picks the token by inverse CDF.
//
// A CTA never waits for work another CTA has yet to start; the only cross-CTA wait is the idle
// wait at the very end (CTAs that ran out of units stay to serve second-pass pieces until every
// sequence is final), which cannot deadlock and is time-limited.
#pragma once
#include "ears_common.cuh"
#include "ears_kernel.cuh"   // finalize_sequence, select_token and their helpers
#include "ears_math.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"

namespace ears {

#ifndef EARS_D_THREADS
#define EARS_D_THREADS 256
#endif
#ifndef EARS_D_CTAS
#define EARS_D_CTAS 3
#endif
constexpr int kDThreads = EARS_D_THREADS;
constexpr int kDWarps = kDThreads / 32;
constexpr int kDCtasPerSm = EARS_D_CTAS;
#ifndef EARS_D_UNROLL
#define EARS_D_UNROLL 8
#endif
constexpr int kDUnroll = EARS_D_UNROLL;            // 16-byte loads in flight per thread
constexpr int kBonusSegBytes = kChunkBytes / kConsumerWarps;   // bytes of the extra row per stored sum (2 KB)

enum DWorkKind : int { kDUnit = 0, kDJob = 1, kDIdle = 2, kDExit = 3 };
struct DWork { int kind; int b; int n; int part; long long unit; };

struct DSmem {
    DWork work[2];                 // alternating by iteration
    float4 red[2][kDWarps];        // per-warp (m, s) of a unit, alternating by iteration
    int abort_flag;
};

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// An ordinary row piece [e0, e1): THREADS threads (tid = 0 .. THREADS-1) stride over it.
// -> the thread's (m, s); ENT: also *w_out = its sum e t (see RowAccT).
template <typename E, int THREADS = kDThreads, bool ENT = false>
__device__ __forceinline__ float2 stream_piece(const E* row, int e0, int e1, bool vec, float c, int tid, float* w_out = nullptr) {
    constexpr int N = Words<E>::N;
    RowAccT<ENT> a;
    acc_open(a);
    if (vec) {
        const uint4* vs = reinterpret_cast<const uint4*>(row + e0);
        const int nvec = (e1 - e0) / N;   // rows and pieces are whole vectors here
        int v = tid;
        for (; v + (kDUnroll - 1) * THREADS < nvec; v += kDUnroll * THREADS) {
            uint4 w[kDUnroll];
#pragma unroll
            for (int j = 0; j < kDUnroll; ++j) w[j] = ld_stream16(vs + v + j * THREADS);
            fold_vectors<E, kDUnroll, ENT>(w, c, a);
        }
        for (; v + THREADS < nvec; v += 2 * THREADS) {   // what is left of a piece: two, then one at a time
            uint4 w[2] = {ld_stream16(vs + v), ld_stream16(vs + v + THREADS)};
            fold_vectors<E, 2, ENT>(w, c, a);
        }
        for (; v < nvec; v += THREADS) {
            uint4 w[1] = {ld_stream16(vs + v)};
            fold_vectors<E, 1, ENT>(w, c, a);
        }
    } else {  // rows that are not 16-byte aligned: element by element
        for (int i = e0 + tid; i < e1; i += THREADS) {
            const float x = load_logit(row + i);
            acc_raise(a, x, c);
            acc_add_one(a, x, c);
        }
    }
    return acc_close(a, c, w_out);
}

// A piece [e0, e1) of the extra target row: warp w takes the segments w, w + kDWarps, ... of
// kBonusSegBytes each, two per round (eight loads in flight per lane), keeps a warp-uniform
// running maximum and stores (sum, reference maximum) of every segment.
// -> the lane's (m, s) relative to the warp's final maximum.
template <typename E>
__device__ __forceinline__ float2 stream_bonus_piece(const E* row, int e0, int e1, bool vec, float c, int warp, int lane,
                                                     BonusSeg* segs /* of the whole row */) {
    constexpr int N = Words<E>::N;
    constexpr int SEG = kBonusSegBytes / (int)sizeof(E);   // entries per segment
    constexpr int VPL = SEG / N / 32;                        // vectors per lane per segment
    constexpr int PN = N / 2;
    RowAcc a;            // the maximum is kept warp-uniform
    acc_open(a);
    for (int ga = e0 + warp * SEG; ga < e1; ga += 2 * kDWarps * SEG) {
        // the loads stay packed (16 bytes per vector) until they are used; rows that are not
        // 16-byte aligned are gathered element by element into the same form
        uint4 w[2][VPL];
        float cm[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int g0 = ga + h * kDWarps * SEG;
            const int cnt = max(0, min(SEG, e1 - g0));
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int k0 = (j * 32 + lane) * N;
                if (vec) {
                    w[h][j] = k0 < cnt ? ld_stream16(row + g0 + k0) : Words<E>::minus_inf();
                } else {
                    w[h][j] = Words<E>::gather(row + g0 + k0, cnt - k0);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) cm[h] = Words<E>::template vmax_all<VPL>(w[h]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            cm[0] = fmaxf(cm[0], __shfl_xor_sync(0xffffffffu, cm[0], off));
            cm[1] = fmaxf(cm[1], __shfl_xor_sync(0xffffffffu, cm[1], off));
        }
        double tot[2];
        float ref[2];   // the fp32 product (running maximum) x c the segment's terms are relative to
        const f32x2 c2 = pack2(c, c);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            acc_raise(a, cm[h], c);
            ref[h] = a.mu;
            const f32x2 nmu2 = pack2(-a.mu, -a.mu);
            f32x2 cs[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                f32x2 p[PN];
                Words<E>::pairs(w[h][j], p);
#pragma unroll
                for (int i = 0; i < PN; i += 2) {
                    cs[0] = add2(cs[0], ex2_pair(fma2(p[i], c2, nmu2)));
                    cs[1] = add2(cs[1], ex2_pair(fma2(p[i + 1], c2, nmu2)));
                }
            }
            a.s[0] = add2(a.s[0], cs[0]);
            a.s[1] = add2(a.s[1], cs[1]);
            float q0, q1;
            unpack2(add2(cs[0], cs[1]), q0, q1);
            tot[h] = (double)(q0 + q1);
        }
        // a lane's few terms add up in fp32; across lanes in fp64 (the running sums of the final
        // draw stay exact to ~1e-9 of the row's mass)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            tot[0] += __shfl_xor_sync(0xffffffffu, tot[0], off);
            tot[1] += __shfl_xor_sync(0xffffffffu, tot[1], off);
        }
        if (lane == 0) {
            segs[ga / SEG] = BonusSeg{tot[0], ref[0], 0.f};
            if (ga + kDWarps * SEG < e1) segs[(ga + kDWarps * SEG) / SEG] = BonusSeg{tot[1], ref[1], 0.f};
        }
    }
    // the draw looks at whole 16 KB chunks: segments of the row's last chunk that lie beyond its
    // end hold no mass
    constexpr int CHUNK = kChunkBytes / (int)sizeof(E);
    const int e_pad = (e1 + CHUNK - 1) / CHUNK * CHUNK;
    for (int g0 = (e1 + SEG - 1) / SEG * SEG + warp * SEG; g0 < e_pad; g0 += kDWarps * SEG)
        if (lane == 0) segs[g0 / SEG] = BonusSeg{0.0, 0.f, 0.f};
    return acc_close(a, c);
}

// A second-pass piece [e0, e1) of the two rows of a rejected position: sums of
// max(0, e_t - e_d Z_t / Z_d) per kSegElems entries; warp w takes groups of four segments and
// keeps the loads of a group (packed, as they come) in flight together.  RESID = false: the
// target row alone, sums of e_t (a bonus token is drawn from P_t).
template <typename E, bool RESID = true>
__device__ __forceinline__ void stream_job_piece(const E* trow, const E* drow, int e0, int e1, bool vec, const RowNorm& rn,
                                                 float c, int warp, int lane, double* seg_out /* of the whole row */) {
    constexpr int N = Words<E>::N;
    constexpr int VPL = kSegElems / N / 32;   // vectors per lane per segment and row
    constexpr int GROUP = VPL >= 2 ? 2 : 4;   // segments per round: 32 registers of loads in flight for either row width
    for (int g0 = e0 + warp * GROUP * kSegElems; g0 < e1; g0 += kDWarps * GROUP * kSegElems) {
        double acc[GROUP];
        if (vec) {
            uint4 wt[GROUP][VPL], wd[GROUP][VPL];
#pragma unroll
            for (int h = 0; h < GROUP; ++h)
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    const int k0 = g0 + h * kSegElems + (j * 32 + lane) * N;
                    if (k0 < e1) {
                        wt[h][j] = ld_stream16(trow + k0);
                        wd[h][j] = RESID ? ld_stream16(drow + k0) : make_uint4(0, 0, 0, 0);
                    } else {
                        wt[h][j] = make_uint4(0, 0, 0, 0);
                        wd[h][j] = make_uint4(0, 0, 0, 0);
                    }
                }
#pragma unroll
            for (int h = 0; h < GROUP; ++h) {
                float a = 0.f;
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    float xt[N], xd[N];
                    Words<E>::unpack(wt[h][j], xt);
                    Words<E>::unpack(wd[h][j], xd);
                    const bool in = g0 + h * kSegElems + (j * 32 + lane) * N < e1;   // whole vectors here
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        const float r = entry_mass<RESID>(xt[i], xd[i], rn, c);
                        if (in) a += r;
                    }
                }
                acc[h] = (double)a;
            }
        } else {
#pragma unroll
            for (int h = 0; h < GROUP; ++h) {
                float a = 0.f;
                for (int j = 0; j < VPL; ++j)
                    for (int i = 0; i < N; ++i) {
                        const int k = g0 + h * kSegElems + (j * 32 + lane) * N + i;
                        if (k < e1) a += entry_mass<RESID>(load_logit(trow + k), RESID ? load_logit(drow + k) : 0.f, rn, c);
                    }
                acc[h] = (double)a;
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
#pragma unroll
            for (int h = 0; h < GROUP; ++h) acc[h] += __shfl_xor_sync(0xffffffffu, acc[h], off);
        if (lane == 0) {
#pragma unroll
            for (int h = 0; h < GROUP; ++h)
                if (g0 + h * kSegElems < e1) seg_out[(g0 + h * kSegElems) / kSegElems] = acc[h];
        }
    }
}

// Named barriers between the streaming warps and the control warp (ids 1..4; 0 is __syncthreads).
// A generation is complete when all kDThreads + 32 threads have arrived (streamers and control).
// (The ids are immediates: with a register operand the compiler reserves all sixteen barriers of
// the SM for one CTA.)
template <int ID> __device__ __forceinline__ void nb_sync_id() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(kDThreads + 32) : "memory"); }
template <int ID> __device__ __forceinline__ void nb_arrive_id() { asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(kDThreads + 32) : "memory"); }
// A(it): ids 1, 2 by parity; B(it): ids 3, 4 by parity
__device__ __forceinline__ void sync_A(int it) { if (it & 1) nb_sync_id<2>(); else nb_sync_id<1>(); }
__device__ __forceinline__ void arrive_A(int it) { if (it & 1) nb_arrive_id<2>(); else nb_arrive_id<1>(); }
__device__ __forceinline__ void sync_B(int it) { if (it & 1) nb_sync_id<4>(); else nb_sync_id<3>(); }
__device__ __forceinline__ void arrive_B(int it) { if (it & 1) nb_arrive_id<4>(); else nb_arrive_id<3>(); }

// Control-warp side of a finished work item: publish and count the piece, and do what falls to
// the CTA that delivered a sequence's last piece.
template <typename E, bool PER_SEQ, bool ENT>
__device__ __forceinline__ void direct_epilogue(const Params& p, const DWork& wk, const float4* red, int lane) {
    const int K = p.K, R = 2 * K + 1, P = p.plan.parts1, P2 = p.plan.parts2;
    if (wk.kind == kDUnit) {
        const long long u = wk.unit;
        const int b = (int)(u / (R * P));
        const int rem = (int)(u % (R * P));
        const int ridx = rem / P, part = rem % P;
        const float c = PER_SEQ ? seq_c(p, b) : p.c;
        const float4 v = red[lane & (kDWarps - 1)];
        float MM = v.x;
#pragma unroll
        for (int off = kDWarps / 2; off > 0; off >>= 1) MM = fmaxf(MM, __shfl_xor_sync(0xffffffffu, MM, off));
        const float2 sw = ENT ? rebase_sum_w(v.x, v.y, v.z, MM, c) : make_float2(rebase_sum(v.x, v.y, MM, c), 0.f);
        float SS = sw.x, WW = sw.y;
#pragma unroll
        for (int off = kDWarps / 2; off > 0; off >>= 1) {
            SS += __shfl_xor_sync(0xffffffffu, SS, off);
            if (ENT) WW += __shfl_xor_sync(0xffffffffu, WW, off);
        }
        int last_b = -1;
        if (lane == 0) {
            p.partial[((size_t)b * R + ridx) * P + part] = make_float2(MM, SS);
            if (ENT) p.partial_w[((size_t)b * R + ridx) * P + part] = WW;
            // two-level count (row, then sequence) keeps same-address atomics rare; the atomics
            // release this piece and acquire the others
            bool row_done = true;
            if (P > 1) row_done = ticket_add(&p.ticket_row[(size_t)b * R + ridx]) == P - 1;
            if (row_done && ticket_add(&p.ticket1[b]) == R - 1) last_b = b;
        }
        last_b = __shfl_sync(0xffffffffu, last_b, 0);
        if (last_b >= 0) {
            // this CTA delivered the sequence's last piece: decide it
            __threadfence();
            const int n = finalize_sequence<E, ENT>(p, last_b, lane);
            __threadfence();
            __syncwarp();
            if (n == K) {
                select_token<E>(p, last_b, n, lane);   // every draft accepted: the extra row's sums are there
            } else if (n >= 0 && lane == 0) {
                const int slot = atomicAdd(&p.heads[3], 1);   // publish for the second pass
                *reinterpret_cast<volatile unsigned long long*>(&p.ready[slot]) =
                    ((unsigned long long)(last_b + 1) << 32) | (unsigned)n;
            }
            if (lane == 0) {   // finalised (valid or not): lets idle CTAs know when to leave
                __threadfence();
                atomicAdd(&p.heads[1], 1);
            }
        }
    } else if (wk.kind == kDJob) {
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = ticket_add(&p.ticket2[wk.b]) == P2 - 1 ? 1 : 0;   // all masses summed
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            __threadfence();
            select_token<E>(p, wk.b, wk.n, lane);
        }
    }
}

// kDThreads streaming threads plus one control warp.  Iteration `it`:
//   control   selects work item it, publishes it in work[it & 1], arrives on barrier A(it); then
//             waits on barrier B(it - 1) for the streamers' result of item it - 1 and runs its
//             epilogue -- while the streamers are already busy with item it;
//   streamers wait on A(it), process item it, leave their per-warp results in red[it & 1],
//             arrive on B(it) and go on.
// A and B alternate between two barrier ids by the parity of `it`; a generation always gets
// exactly one arrival from every streaming thread and every control lane, on every path.
template <typename E, bool PER_SEQ, bool ENT>
__global__ void __launch_bounds__(kDThreads + 32, kDCtasPerSm) ears_direct_kernel(const Params p) {
    __shared__ DSmem sm;
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1, cpp = p.plan.cpp1, P2 = p.plan.parts2;
    const bool vec = p.plan.use_tma != 0;   // rows are 16-byte aligned
    const int chunks_per_row = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    const long long total_units = (long long)p.B * R * P;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const E* tbase = reinterpret_cast<const E*>(p.t);
    const E* dbase = reinterpret_cast<const E*>(p.d);

    if (tid == 0) trace_mark(0, 0);
    clear_next_counters(p);
    if (tid == 0) sm.abort_flag = 0;
    __syncthreads();

    if (warp == kDWarps) {
        // =============================== control warp
        long long u_ahead = 0;   // the queue index of the next unit, fetched one unit ahead (lane 0)
        if (lane == 0) u_ahead = atomicAdd(&p.heads[0], 1);
        bool stats_done = false, all_final = false, piece_last = false;
        int cursor = 0;
        unsigned long long wait_t0 = 0;
        DWork prev{kDIdle, 0, 0, 0, 0};
        for (int it = 0;; ++it) {
            DWork wk{kDIdle, 0, 0, 0, 0};
            bool prev_done = it == 0;
            for (;;) {
                // Published sequences form a queue of (sequence, piece) served by every CTA in order:
                // each lane looks at one of the next 32 published slots; the first with pieces left
                // is tried with one atomic.  Pieces and units alternate while both exist, so that a
                // unit whose ticket this CTA already holds does not wait behind a long run of pieces.
                bool again = false;
                if (!(piece_last && !stats_done)) {
                    const int slot = cursor + lane;
                    unsigned long long e = 0;
                    int taken = P2;
                    if (slot < p.B) {
                        e = *reinterpret_cast<volatile unsigned long long*>(&p.ready[slot]);
                        taken = *reinterpret_cast<volatile int*>(&p.job_ctr[slot]);
                    }
                    const unsigned open = __ballot_sync(0xffffffffu, e != 0 && taken < P2);
                    const unsigned done = __ballot_sync(0xffffffffu, e != 0 && taken >= P2);
                    cursor += done == 0xffffffffu ? 32 : __ffs(~done) - 1;   // skip leading exhausted slots
                    again = open != 0;
                    if (open) {
                        const int L = __ffs(open) - 1;
                        int piece = P2;
                        if (lane == L) piece = atomicAdd(&p.job_ctr[slot], 1);
                        piece = __shfl_sync(0xffffffffu, piece, L);
                        if (piece < P2) {
                            const unsigned long long el = __shfl_sync(0xffffffffu, e, L);
                            wk = DWork{kDJob, (int)(el >> 32) - 1, (int)(unsigned)el, piece, 0};
                        }
                    }
                }
                piece_last = wk.kind == kDJob;
                if (wk.kind == kDIdle && !stats_done) {
                    const long long u = __shfl_sync(0xffffffffu, u_ahead, 0);
                    if (u >= total_units) {
                        stats_done = true;
                    } else {
                        if (lane == 0) u_ahead = atomicAdd(&p.heads[0], 1);
                        wk = DWork{kDUnit, 0, 0, 0, u};
                    }
                }
                if (wk.kind != kDIdle) break;
                // Nothing to hand out right now.  First finish the previous item (its sequence may
                // be waiting for exactly that), then look again.
                if (!prev_done) {
                    sync_B(it - 1);
                    if (lane == 0) trace_mark(15, 1);
                    direct_epilogue<E, PER_SEQ, ENT>(p, prev, sm.red[(it - 1) & 1], lane);
                    if (lane == 0) trace_mark(16, 1);
                    prev_done = true;
                    continue;
                }
                if (again) continue;   // pieces exist, another CTA was quicker
                // No units left and no piece to claim: stay until every sequence of the batch has been
                // finalised (by whichever CTA) and a look after that found no piece either.  A
                // sequence is finalised by a CTA that already holds its last unit and waits for
                // nobody, so this cannot deadlock; it is bounded like every other wait.
                if (all_final) { wk.kind = kDExit; break; }
                int fin = 0;
                if (lane == 0) {
                    fin = *reinterpret_cast<volatile int*>(&p.heads[1]) >= p.B ? 1 : 0;
                    if (!fin) {
                        const unsigned long long now = global_timer_ns();
                        if (wait_t0 == 0) wait_t0 = now;
                        else if (now - wait_t0 > kIdleLimitNs) fin = -1;
                        __nanosleep(100);
                    }
                }
                fin = __shfl_sync(0xffffffffu, fin, 0);
                if (fin < 0) { if (lane == 0) sm.abort_flag = 1; wk.kind = kDExit; break; }
                if (fin > 0) { all_final = true; __threadfence(); }
            }
            if (lane == 0) sm.work[it & 1] = wk;
            __threadfence_block();
            __syncwarp();
            if (lane == 0) trace_mark(10 + wk.kind, (int)wk.unit);
            arrive_A(it);                                    // A(it): the item is published
            if (!prev_done) {
                sync_B(it - 1);                               // B(it - 1): the previous item's results are in
                if (lane == 0) trace_mark(15, 0);
                direct_epilogue<E, PER_SEQ, ENT>(p, prev, sm.red[(it - 1) & 1], lane);
                if (lane == 0) trace_mark(16, 0);
            }
            if (wk.kind == kDExit) break;
            prev = wk;
        }
    } else {
        // =============================== streaming warps
        for (int it = 0;; ++it) {
            sync_A(it);                                      // A(it)
            const DWork wk = sm.work[it & 1];
            if (wk.kind == kDExit) break;
            if (wk.kind == kDUnit) {
                const long long u = wk.unit;
                const int b = (int)(u / (R * P));
                const int rem = (int)(u % (R * P));
                const int ridx = rem / P, part = rem % P;
                const bool bonus = ridx == 2 * K;
                const E* row = bonus ? tbase + (size_t)target_row(b, K, K) * V
                                     : ((ridx & 1) ? dbase + (size_t)draft_row(b, ridx >> 1, K) * V
                                                   : tbase + (size_t)target_row(b, ridx >> 1, K) * V);
                const float c = PER_SEQ ? seq_c(p, b) : p.c;
                const int e0 = min(V, part * cpp * CHUNK_ELEMS);
                const int e1 = min(V, min(chunks_per_row, (part + 1) * cpp) * CHUNK_ELEMS);
                float2 ms;
                float wv = 0.f;   // ENT: the thread's sum e t (target rows of positions only; the others do not need it)
                if (bonus) ms = stream_bonus_piece<E>(row, e0, e1, vec, c, warp, lane, bonus_segs(p, b));
                else if (ENT && !(ridx & 1)) ms = stream_piece<E, kDThreads, true>(row, e0, e1, vec, c, tid, &wv);
                else ms = stream_piece<E>(row, e0, e1, vec, c, tid);
                // (max, sum) of the warp: the maximum first, one rescale per thread, then a sum
                float M = ms.x;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
                const float2 sw = ENT ? rebase_sum_w(ms.x, ms.y, wv, M, c) : make_float2(rebase_sum(ms.x, ms.y, M, c), 0.f);
                float S = sw.x, W = sw.y;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    S += __shfl_xor_sync(0xffffffffu, S, off);
                    if (ENT) W += __shfl_xor_sync(0xffffffffu, W, off);
                }
                if (lane == 0) sm.red[it & 1][warp] = make_float4(M, S, W, 0.f);
            } else {
                // second pass: one piece of the two rows of sequence b's first rejected position n
                __threadfence();
                const int b = wk.b, n = wk.n;
                const float c = PER_SEQ ? seq_c(p, b) : p.c;
                const E* trow = tbase + (size_t)target_row(b, n, K) * V;
                const E* drow = dbase + (size_t)draft_row(b, n, K) * V;
                const float2 st = __ldcg(&p.rowstat[(size_t)b * R + 2 * n]);
                const float2 sd = __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]);
                const RowNorm rn = make_rownorm(st, sd);
                const int e0 = min(V, wk.part * p.plan.job_elems), e1 = min(V, e0 + p.plan.job_elems);
                stream_job_piece<E>(trow, drow, e0, e1, vec, rn, c, warp, lane, seg_sums(p, b));
            }
            __threadfence();   // segment sums and results: visible before the control warp counts the piece
            arrive_B(it);                                    // B(it): this item's results are in shared / global memory
        }
    }
    __syncthreads();
    if (tid == 0) trace_mark(6, 0);
    if (tid == 0 && sm.abort_flag) atomicOr(&p.heads[2], kDevTimeout);
}

}  // namespace ears
