// The verification step as one persistent kernel.
//
// Work is cut into "units" (a piece of one logits row) that CTAs pull from an atomic queue,
// sequence by sequence.  Inside a CTA:
//
//   loader warp     pulls units and streams them into a ring of shared-memory slots with 1-D
//                   bulk asynchronous copies completing on mbarriers (element-wise copies when
//                   the data is not 16-byte aligned); also serves the second pass (below);
//   8 consumer      keep a running (max, sum exp2) per thread over the slots [softmax
//   warps           statistics, Sec. 3.1] and reduce them per unit; for the extra target row K
//                   they also leave per-warp chunk sums behind;
//   epilogue warp   publishes the pieces of rows and counts them with atomic tickets (per row,
//                   then per sequence), so that consumers never wait at the end of a unit;
//   sequence warp   for a sequence whose last piece this CTA delivered: merges the pieces, forms
//                   P_t(x), P_d(x), max P_t = 1/Z_t, draws U_k, decides every position (Sec. 3.2
//                   with the guards of Sec. 3.3 item 2) and scans for the first rejection
//                   (Sec. 3.1).  If every draft was accepted the bonus token is drawn at once
//                   from the chunk sums of row K.  Otherwise the sequence is published for a
//                   second pass over the two rows of the rejected position: all CTAs serve
//                   those rows in pieces (they were streamed moments ago and are mostly still
//                   in L2), consumers turn them into segment sums of max(0, P_t - P_d), and the
//                   CTA that delivers the last piece picks the token by inverse CDF.
//
// A CTA never waits for work another CTA has yet to start; the only cross-CTA wait is the idle
// wait at the very end (see the loader), which cannot deadlock.  Every wait is bounded.
#pragma once
#include "ears_common.cuh"
#include "ears_philox.cuh"
#include "ears_pipeline.cuh"
#include "ears_math.cuh"

namespace ears {

enum ChunkKind : int { kStats = 0, kFinal = 1, kEnd = 4 };
enum MsgKind : int { kMsgPiece = 0, kMsgJobPiece = 1, kMsgExit = 3, kMsgNone = 6 };

struct alignas(16) StageMeta {   // 32 bytes: two 16-byte shared-memory accesses
    int kind;    // ChunkKind
    int id;      // unit index (statistics) or sequence index (final-token rows)
    int nelem;   // valid elements per row in the slot
    int flags;   // bit 0: first chunk of the unit / row, bit 1: last chunk
    int elem0;   // index of the slot's first element within its row
    int aux;     // statistics: 1 for the extra target row; final-token rows: position n
    float c;     // log2(e) / temperature of the slot's sequence
    int pad;
};

struct Msg { int kind, a, b, c; };

// Single-producer single-consumer ring in shared memory.  One lane pushes, one lane pops.
template <int CAP>
struct Mailbox {
    volatile int head, tail;
    volatile int slot[CAP][4];

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
        slot[t % CAP][0] = m.kind; slot[t % CAP][1] = m.a; slot[t % CAP][2] = m.b; slot[t % CAP][3] = m.c;
        __threadfence_block();
        tail = t + 1;
        return true;
    }
    __device__ __forceinline__ bool try_pop(Msg& m) {
        const int h = head;
        if (h == tail) return false;
        __threadfence_block();
        m.kind = slot[h % CAP][0]; m.a = slot[h % CAP][1]; m.b = slot[h % CAP][2]; m.c = slot[h % CAP][3];
        __threadfence_block();
        head = h + 1;
        return true;
    }
    // Waits for at least one message; returns how many (<= 32) are ready starting at *first,
    // or -1 when the block is aborting or the time limit passed.  Called by one lane.
    __device__ __forceinline__ int wait_batch(int* first, volatile int* abort_flag, unsigned long long limit_ns) {
        unsigned long long t0 = 0;
        for (unsigned spin = 0;; ++spin) {
            const int h = head, n = tail - h;
            if (n > 0) { *first = h; return n < 32 ? n : 32; }
            if ((spin & 15u) == 15u) {
                if (*abort_flag) return -1;
                unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > limit_ns) { *abort_flag = 1; return -1; }
            }
            __nanosleep(50);
        }
    }
    __device__ __forceinline__ Msg peek(int index) const {
        return Msg{slot[index % CAP][0], slot[index % CAP][1], slot[index % CAP][2], slot[index % CAP][3]};
    }
    __device__ __forceinline__ void release(int new_head) { __threadfence_block(); head = new_head; }

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
            __nanosleep(50);
        }
    }
};

// consumer warp 0 -> epilogue warp
constexpr int kEpiCap = 64;
// epilogue warp -> sequence warp: only the exit message
constexpr int kSeqCap = 4;
// Ends of units are handed to the epilogue warp through a ring of slots: each consumer warp
// drops its (m, s) there and arrives on the slot's barrier, so no consumer ever waits for
// another at the end of a unit.  Consumer warps are at most one pipeline ring apart, and
// warp 0 holds back while kUnitGuard ends are unread, hence the slots cannot be overrun.
constexpr int kUnitSlots = 16;
constexpr int kUnitGuard = 8;
// A warp that is idle by design (the epilogue and sequence warps between messages, a CTA that ran
// out of units and stays to help) may wait for as long as the rest of the kernel runs.  The largest
// input that fits this GPU's 180 GB of HBM streams in under 30 ms, so half a second is a limit no
// healthy launch comes near, and a slip in the hand-over logic costs the GPU half a second, not half a minute.
constexpr unsigned long long kIdleLimitNs = 500000000ull;

template <int STAGES>
struct PipeSmem {
    alignas(128) unsigned char buf[STAGES][kChunkBytes];
    alignas(8) uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t unit_bar[kUnitSlots];
    StageMeta meta[STAGES];
    float4 scratch[kUnitSlots][kConsumerWarps];   // (m, s, sum e t, -) of each consumer warp at a unit's end
    volatile int units_read;   // unit ends the epilogue warp has taken out of the slots
    Mailbox<kEpiCap> epi;
    Mailbox<kSeqCap> seq;
    int abort_flag;
};

// Consumer warp 0, one lane: announce the end of a unit, holding back while too many are unread.
template <int STAGES>
__device__ __forceinline__ void push_unit_end(PipeSmem<STAGES>& sm, const Msg& m) {
    unsigned long long t0 = 0;
    for (unsigned spin = 0; m.c - sm.units_read >= kUnitGuard; ++spin) {
        if ((spin & 15u) == 15u) {
            if (sm.abort_flag) return;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) { sm.abort_flag = 1; return; }
        }
        __nanosleep(40);
    }
    sm.epi.push(m, &sm.abort_flag, kWaitLimitNs);
}

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
    for (int i = lane; i < n; i += 32) o[i] = ld_elem(src + i);
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
                                            const E* src0, const E* src1, int lane, uint64_t policy) {
    if (lane == 0) sm.meta[stage] = mt;
    const uint32_t bytes = (uint32_t)mt.nelem * (uint32_t)sizeof(E);
    if (use_tma) {
        if (lane == 0) {
            if (bytes == 0 || !src0) {
                mbar_arrive(&sm.full[stage]);
            } else {
                mbar_arrive_expect_tx(&sm.full[stage], src1 ? 2 * bytes : bytes);
                if (policy) {
                    bulk_load_hint(sm.buf[stage], src0, bytes, &sm.full[stage], policy);
                    if (src1) bulk_load_hint(sm.buf[stage] + kChunkBytes / 2, src1, bytes, &sm.full[stage], policy);
                } else {
                    bulk_load(sm.buf[stage], src0, bytes, &sm.full[stage]);
                    if (src1) bulk_load(sm.buf[stage] + kChunkBytes / 2, src1, bytes, &sm.full[stage]);
                }
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
// Running (m, s) of one thread over its share of a staged chunk, in the RowAcc form: one
// multiply-add, one exp2 and one addition per entry, the first and the last on pairs of entries.
// Warp w owns the w-th eighth of the slot (contiguous), lane-interleaved in 16-byte vectors.
//
// BONUS (the extra target row K): the maximum is kept warp-uniform and the warp also emits the sum
// of its eighth of the chunk together with the reference the terms were taken against.  If every
// draft token turns out to be accepted, the final token is drawn from exactly these sums and the
// row is not read again.
template <typename E, bool BONUS, bool ENT>
__device__ __forceinline__ void chunk_stats(const unsigned char* buf, int nelem, int warp, int lane, float c,
                                            RowAccT<ENT>& a, BonusSeg* warp_chunk_out) {
    constexpr int N = Words<E>::N, PN = N / 2;
    constexpr int VECS = kChunkBytes / 16 / kConsumers;  // 16-byte vectors per thread per chunk
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    uint4 w[VECS];
#pragma unroll
    for (int j = 0; j < VECS; ++j) w[j] = reinterpret_cast<const uint4*>(buf)[(warp * VECS + j) * 32 + lane];
    if (nelem < CHUNK_ELEMS) {  // ragged last chunk of a row: mask what lies beyond it
#pragma unroll
        for (int j = 0; j < VECS; ++j) w[j] = Words<E>::mask_tail(w[j], nelem - ((warp * VECS + j) * 32 + lane) * N);
    }
    if (!BONUS) {
        fold_vectors<E, VECS, ENT>(w, c, a);
        return;
    }
    float cm = Words<E>::template vmax_all<VECS>(w);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, off));
    acc_raise(a, cm, c);   // warp-uniform
    const f32x2 c2 = pack2(c, c), nmu2 = pack2(-a.mu, -a.mu);
    f32x2 cs[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
    for (int j = 0; j < VECS; ++j) {
        f32x2 p[PN];
        Words<E>::pairs(w[j], p);
#pragma unroll
        for (int i = 0; i < PN; i += 2) {
            cs[0] = add2(cs[0], ex2_pair(fma2(p[i], c2, nmu2)));
            cs[1] = add2(cs[1], ex2_pair(fma2(p[i + 1], c2, nmu2)));
        }
    }
    a.s[0] = add2(a.s[0], cs[0]);
    a.s[1] = add2(a.s[1], cs[1]);
    // a lane's few terms add up in fp32; across lanes in fp64, so that the running sums of the
    // final draw stay exact to ~1e-9 of the row's mass
    float q0, q1;
    unpack2(add2(cs[0], cs[1]), q0, q1);
    double tot = (double)(q0 + q1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, off);
    if (lane == 0) *warp_chunk_out = BonusSeg{tot, a.mu, 0.f};
}

// Sums of kSegElems-element segments of a staged chunk; warp w takes segments w, w+8, ...
// A lane adds its few masses in fp32; lanes are added in fp64.
template <typename E, bool RESID>
__device__ __forceinline__ void chunk_segments(const unsigned char* bt, const unsigned char* bd, int nelem,
                                               int warp, int lane, const RowNorm& rn, float c, double* seg_out) {
    constexpr int N = Vec<E>::N;
    constexpr int VECS = kSegElems / (32 * N);  // 16-byte vectors per lane per segment
    constexpr int FULL_ELEMS = (RESID ? kChunkBytes / 2 : kChunkBytes) / (int)sizeof(E);
    constexpr int SEGS = FULL_ELEMS / kSegElems / kConsumerWarps;  // segments per warp in a full slot
    if (SEGS >= 1 && nelem == FULL_ELEMS) {
        // full slot: all of the warp's segments at once, so that their loads, exponentials and
        // shuffle trees overlap instead of running one after the other
        double acc[SEGS > 0 ? SEGS : 1];
#pragma unroll
        for (int g = 0; g < SEGS; ++g) {
            float a = 0.0f;
#pragma unroll
            for (int j = 0; j < VECS; ++j) {
                const int vec = (g * kConsumerWarps + warp) * (kSegElems / N) + j * 32 + lane;
                float xt[N], xd[N];
                Vec<E>::load(bt, vec, xt);
                if (RESID) Vec<E>::load(bd, vec, xd);
#pragma unroll
                for (int i = 0; i < N; ++i) a += entry_mass<RESID>(xt[i], RESID ? xd[i] : 0.f, rn, c);
            }
            acc[g] = (double)a;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
#pragma unroll
            for (int g = 0; g < SEGS; ++g) acc[g] += __shfl_xor_sync(0xffffffffu, acc[g], off);
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < SEGS; ++g) seg_out[g * kConsumerWarps + warp] = acc[g];
        }
        return;
    }
    const int nseg = (nelem + kSegElems - 1) / kSegElems;
    for (int sgm = warp; sgm < nseg; sgm += kConsumerWarps) {
        float a = 0.0f;
#pragma unroll
        for (int j = 0; j < VECS; ++j) {
            const int vec = sgm * (kSegElems / N) + j * 32 + lane;
            float xt[N], xd[N];
            Vec<E>::load(bt, vec, xt);
            if (RESID) Vec<E>::load(bd, vec, xd);
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const float r = entry_mass<RESID>(xt[i], RESID ? xd[i] : 0.f, rn, c);
                if (vec * N + i < nelem) a += r;
            }
        }
        double acc = (double)a;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) seg_out[sgm] = acc;
    }
}

// ---- epilogue warp: decisions -----------------------------------------------------
// Merges the pieces of all 2K+1 rows, writes (m, Z) per row, decides every position
// (Sec. 3.2 steps 1-5 with the guards of Sec. 3.3 item 2) and writes the accepted
// prefix (Sec. 3.1).  Returns the accepted length n, or -1 for an invalid sequence.
template <typename E, bool ENT>
__device__ int finalize_sequence(const Params& p, int b, int lane) {
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1;
    const E* t = reinterpret_cast<const E*>(p.t);
    const E* d = reinterpret_cast<const E*>(p.d);
    const float cb = seq_c(p, b);
    const double Tb = seq_temperature(p, b), betab = seq_beta(p, b);
    // `bad`: something that invalidates the sequence wherever it is; with stop_first only what lies
    // at or before the first rejection counts [Sec. 3.1: later draft tokens are discarded anyway],
    // tracked per position in `stop` (the first position that is rejected or unusable ends the scan).
    const bool stop_first = p.stop_first != 0;
    bool bad = !seq_params_ok(Tb, betab);
    // Dependent round trips through L2 are what this function costs (it runs on one warp while the
    // sequence's CTAs wait for nobody, but every sequence passes through it), so loads go out in
    // batches and as early as their addresses are known: the draft tokens first, then the pieces of
    // the rows, then the tokens' logits; with at most 32 rows the rows' statistics then travel between
    // lanes by shuffle instead of through memory.
    const bool rows_fit = R <= 32;
    int tok_early = -1;
    if (rows_fit && lane < K) tok_early = p.x[(size_t)b * K + lane];
    float m_mine = -INFINITY, s_mine = 0.0f, w_mine = 0.0f;   // rows_fit: row `lane`
    for (int r = lane; r < R; r += 32) {
        float m = -INFINITY, s = 0.0f;
        const float2* pp = p.partial + ((size_t)b * R + r) * P;
        for (int i0 = 0; i0 < P; i0 += 8) {
            float2 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = i0 + i < P ? __ldcg(pp + i0 + i) : make_float2(-INFINITY, 0.f);
#pragma unroll
            for (int i = 0; i < 8; ++i) merge_ms(m, s, v[i].x, v[i].y, cb);
        }
        if (!rowstat_ok(m, s) && !stop_first) bad = true;
        p.rowstat[(size_t)b * R + r] = make_float2(m, s);
        float w = 0.f;
        if (ENT && !(r & 1) && r < 2 * K) {
            // sum e t of a target row: its pieces brought to the row maximum (known now)
            const float* pw = p.partial_w + ((size_t)b * R + r) * P;
            for (int i0 = 0; i0 < P; i0 += 8) {
                float2 v[8];
                float q[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    v[i] = i0 + i < P ? __ldcg(pp + i0 + i) : make_float2(-INFINITY, 0.f);
                    q[i] = i0 + i < P ? __ldcg(pw + i0 + i) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) w += rebase_sum_w(v[i].x, v[i].y, q[i], m, cb).y;
            }
            p.roww[(size_t)b * R + r] = w;
        }
        m_mine = m; s_mine = s; w_mine = w;
    }
    float lt_early = 0.f, ld_early = 0.f;
    if (rows_fit && lane < K && tok_early >= 0 && tok_early < V) {
        lt_early = load_logit(t + (size_t)target_row(b, lane, K) * V + tok_early);
        ld_early = load_logit(d + (size_t)draft_row(b, lane, K) * V + tok_early);
    }
    __syncwarp();
    int first_reject = K;
    bool stopped_on_bad = false;
    for (int k0 = 0; k0 < K; k0 += 32) {
        const int k = k0 + lane;
        bool reject = false, posbad = false;
        // the statistics of this position's two rows: from the lanes that merged them, or from memory
        float2 st, sd;
        float wt = 0.f;
        if (rows_fit) {
            const int src = k < K ? 2 * k : 0;
            st = make_float2(__shfl_sync(0xffffffffu, m_mine, src), __shfl_sync(0xffffffffu, s_mine, src));
            sd = make_float2(__shfl_sync(0xffffffffu, m_mine, src + 1), __shfl_sync(0xffffffffu, s_mine, src + 1));
            if (ENT) wt = __shfl_sync(0xffffffffu, w_mine, src);
        } else if (k < K) {
            st = __ldcg(&p.rowstat[(size_t)b * R + 2 * k]);
            sd = __ldcg(&p.rowstat[(size_t)b * R + 2 * k + 1]);
            if (ENT) wt = __ldcg(&p.roww[(size_t)b * R + 2 * k]);
        }
        if (k < K) {
            const int tok = rows_fit ? tok_early : p.x[(size_t)b * K + k];
            posbad = tok < 0 || tok >= V || !rowstat_ok(st.x, st.y) || !rowstat_ok(sd.x, sd.y);
            if (tok < 0 || tok >= V) {
                if (!stop_first) bad = true;
            } else {
                const double lt = (double)(rows_fit ? lt_early : load_logit(t + (size_t)target_row(b, k, K) * V + tok));
                const double ld = (double)(rows_fit ? ld_early : load_logit(d + (size_t)draft_row(b, k, K) * V + tok));
                const double U = uniform_accept(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)k);
                double unc = -1.0;   // < 0: the printed measure, 1 - max P_t
                if (ENT) {
                    const double H = row_entropy(st.y, wt);
                    if (p.entropy) p.entropy[(size_t)b * K + k] = H;
                    if (p.unc_entropy) unc = entropy_uncertainty(H, V);
                }
                const Decision dc = decide_position(lt, ld, st, sd, Tb, betab, U, unc);
                reject = !dc.accept;
                const size_t i = (size_t)b * K + k;
                p.pt_tok[i] = dc.pt;
                p.pd_tok[i] = dc.pd;
                p.max_pt[i] = dc.maxp;
                p.cls[i] = dc.cls;
            }
        }
        const unsigned rej = __ballot_sync(0xffffffffu, stop_first ? (reject || posbad) : reject);
        const unsigned pb = __ballot_sync(0xffffffffu, posbad);
        if (rej != 0 && first_reject == K) {
            first_reject = k0 + __ffs(rej) - 1;
            stopped_on_bad = ((pb >> (__ffs(rej) - 1)) & 1u) != 0;
        }
    }
    if (stop_first) {
        if (stopped_on_bad) bad = true;
        if (first_reject == K) {   // everything accepted: now the extra target row matters too
            const float2 sb = __ldcg(&p.rowstat[(size_t)b * R + 2 * K]);
            if (!rowstat_ok(sb.x, sb.y)) bad = true;
        }
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
        return -1;
    }
    for (int j = lane; j <= K; j += 32) ot[j] = j < first_reject ? p.x[(size_t)b * K + j] : -1;
    if (lane == 0) p.out_len[b] = first_reject;
    // what this sequence decided: the accepted prefix and, if there is one, the first rejection
    // (each lane reads back the classes it wrote itself above)
    const uint8_t* cl = p.cls + (size_t)b * K;
    count_decisions(p.heads, min(first_reject + 1, K), lane, [cl](int k) { return (int)cl[k]; });
    return first_reject;
}

// ---- epilogue warp: final token ---------------------------------------------------
// Slow whole-row draw from P_t by one warp (used only if a residual has no mass).
template <typename E>
__device__ int warp_sample_pt_slow(const E* row, int V, const RowNorm& rn, float c, double u, int lane, double* S_out) {
    const int per = (V + 31) / 32;
    const int v0 = min(V, lane * per), v1 = min(V, v0 + per);
    double loc = 0.0;
    for (int v = v0; v < v1; ++v) loc += (double)entry_mass<false>(load_logit(row + v), 0.f, rn, c);
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
            const double r = (double)entry_mass<false>(load_logit(row + v), 0.f, rn, c);
            if (r > 0.0) lastpos = v;
            cum += r;
            if (target < cum && r > 0.0) { tok = v; break; }
        }
        if (tok < 0) tok = lastpos;
    }
    *S_out = S;
    return __shfl_sync(0xffffffffu, tok, L);
}

// Last level of the inverse-CDF pick: entries [base, base + count) of the row(s) are read again,
// their masses recomputed (same bits as in the streaming pass) and scanned in fp64 for the
// smallest j with tin < running sum.  If rounding hides the crossing, the last entry with
// positive mass is taken.  One warp; count <= 128 * N entries, all loaded up front so that the
// pick costs one memory round trip; returns the token (or -1 if the range has no mass).
template <typename E>
__device__ int pick_in_range(const E* trow, const E* drow, bool resid, const RowNorm& rn, float c,
                             int base, int count, double tin, int V, int lane) {
    constexpr int N = Vec<E>::N;
    constexpr int ROUNDS = 4;  // 4 x 32 lanes x N entries cover the largest range (an eighth of a slot)
    float mass[ROUNDS][N];
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const int k = (j * 32 + lane) * N + i;
            float xt = -INFINITY, xd = -INFINITY;
            const bool valid = k < count && base + k < V;
            if (valid) {
                xt = load_logit(trow + base + k);
                if (resid) xd = load_logit(drow + base + k);
            }
            mass[j][i] = !valid ? 0.f : (resid ? entry_mass<true>(xt, xd, rn, c) : entry_mass<false>(xt, 0.f, rn, c));
        }
    double run = 0.0;
    int found = -1, lastpos = -1;
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
        if (found >= 0 || j * 32 * N >= count) break;
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

// First level: `count` non-negative sums, value(i) for i in [0, count), evaluated by the
// caller-supplied functor (fp64).  Finds the first index whose running sum exceeds u * S and
// returns it with the running sum before it; S is the total.  One warp, lanes own contiguous
// blocks; loads are batched so that a block costs a few memory round trips, not one per entry.
template <typename F>
__device__ int pick_block(F value, int count, double u, int lane, double* S_out, double* before_out) {
    const int per = (count + 31) / 32;
    const int g0 = min(count, lane * per), g1 = min(count, g0 + per);
    double loc = 0.0;
    for (int g = g0; g < g1; g += 8) {
        double v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = g + i < g1 ? value(g + i) : 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) loc += v[i];
    }
    const double inc = warp_inclusive_scan(loc, lane);
    const double S = __shfl_sync(0xffffffffu, inc, 31);
    *S_out = S;
    if (!(S > 0.0)) { *before_out = 0.0; return -1; }
    const double target = u * S;
    const unsigned hit = __ballot_sync(0xffffffffu, target < inc && loc > 0.0);
    const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.0);
    const int L = hit ? __ffs(hit) - 1 : 31 - __clz(pos);
    const double excl_L = __shfl_sync(0xffffffffu, inc - loc, L);
    const int gl0 = __shfl_sync(0xffffffffu, g0, L), gl1 = __shfl_sync(0xffffffffu, g1, L);
    int seg = -1, lastseg = gl0;
    double before = excl_L, before_last = excl_L, run = excl_L;
    for (int gb = gl0; gb < gl1 && seg < 0; gb += 32) {  // lane L's block, 32 sums at a time
        const int g = gb + lane;
        const double v = g < gl1 ? value(g) : 0.0;
        const double incl = warp_inclusive_scan(v, lane);
        const unsigned h = __ballot_sync(0xffffffffu, v > 0.0 && target < run + incl);
        const unsigned ps = __ballot_sync(0xffffffffu, v > 0.0);
        if (ps) {
            const int ll = 31 - __clz(ps);
            lastseg = gb + ll;
            before_last = run + __shfl_sync(0xffffffffu, incl - v, ll);
        }
        if (h) {
            const int l1 = __ffs(h) - 1;
            seg = gb + l1;
            before = run + __shfl_sync(0xffffffffu, incl - v, l1);
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (seg < 0) { seg = lastseg; before = before_last; }
    *before_out = before;
    return seg;
}

// Final token of sequence b (accepted length n): token = smallest j with u*S < C_j over the
// masses of the row(s).  The sums come from the second pass (n < K: residual) or, when every
// draft was accepted, from what the statistics pass left behind for the extra target row.
template <typename E>
__device__ void select_token(const Params& p, int b, int n, int lane) {
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, V = p.V, R = 2 * K + 1, nseg = p.plan.nseg;
    const float cb = seq_c(p, b);
    const bool resid = n < K;
    const E* trow = reinterpret_cast<const E*>(p.t) + (size_t)target_row(b, n, K) * V;
    const E* drow = reinterpret_cast<const E*>(p.d) + (size_t)draft_row(b, resid ? n : 0, K) * V;
    const float2 st = __ldcg(&p.rowstat[(size_t)b * R + (resid ? 2 * n : 2 * K)]);
    const float2 sd = resid ? __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]) : make_float2(0.f, 1.f);
    const RowNorm rn = make_rownorm(st, sd);
    const double u = uniform_final(p.seed, p.offset, (uint32_t)(p.b_first + b), (uint32_t)K);
    double S = 0.0, before = 0.0;
    int seg, seg_elems;
    if (resid) {
        const double* ss = seg_sums(p, b);
        seg = pick_block([ss](int g) { return __ldcg(ss + g); }, nseg, u, lane, &S, &before);
        seg_elems = kSegElems;
    } else {
        // one entry per (chunk, consumer warp) of the extra row: (sum, reference of its terms)
        const int chunks = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
        const BonusSeg* bs = bonus_segs(p, b);
        const double mc = (double)rn.mt * (double)cb;   // exact: two fp32 factors
        seg = pick_block([bs, mc](int g) {
                  const double sum = __ldcg(&bs[g].sum);
                  const float mu = __ldcg(&bs[g].mu);
                  // the terms were exp2(l c - mu): bring the sum to the row's own maximum (fp64: no new error)
                  return sum > 0.0 ? sum * exp2((double)mu - mc) : 0.0;
              }, chunks * kConsumerWarps, u, lane, &S, &before);
        seg_elems = CHUNK_ELEMS / kConsumerWarps;
    }
    int tok;
    double S_used = S;
    if (seg < 0 || !(S * rn.izt >= kTinyMass)) {
        // a rejection implies residual mass; if rounding erased it, draw from P_t instead
        tok = warp_sample_pt_slow<E>(trow, V, rn, cb, u, lane, &S_used);
    } else {
        tok = pick_in_range<E>(trow, drow, resid, rn, cb, seg * seg_elems, seg_elems, u * S - before, V, lane);
    }
    if (lane == 0) {
        p.out_tok[(size_t)b * (K + 1) + n] = tok;
        p.resid[b] = S_used * rn.izt;
    }
}

// ---- the kernel -------------------------------------------------------------------
// PER_SEQ: the call carries per-sequence temperatures, so log2(e)/T comes with every slot;
// otherwise it is the kernel parameter (kept apart: the consumers' code is sensitive to it).
template <typename E, int STAGES, bool PER_SEQ, bool ENT>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) ears_verify_kernel(const Params p) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = PipeSmem<STAGES>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    constexpr int CHUNK_ELEMS = kChunkBytes / (int)sizeof(E);
    const int K = p.K, R = 2 * K + 1, V = p.V, P = p.plan.parts1, cpp = p.plan.cpp1;
    const bool use_tma = p.plan.use_tma != 0;
    const int chunks_per_row = (V + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    const long long total_units = (long long)p.B * R * P;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const E* tbase = reinterpret_cast<const E*>(p.t);
    const E* dbase = reinterpret_cast<const E*>(p.d);

    clear_next_counters(p);
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm.full[s], use_tma ? 1u : 32u);
            mbar_init(&sm.empty[s], kConsumerWarps);
        }
        for (int s = 0; s < kUnitSlots; ++s) mbar_init(&sm.unit_bar[s], kConsumerWarps);
        sm.units_read = 0;
        sm.epi.init();
        sm.seq.init();
        sm.abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();

    if (warp == kLoaderWarp) {
        // =============================== loader warp
        uint32_t q = 0;
        bool ok = true, stats_done = false;
        // The queue index of the next unit is fetched one unit ahead (lane 0 holds it) so that the
        // round trip of the atomic overlaps with streaming the current unit.
        long long u_ahead = 0;
        if (lane == 0) u_ahead = atomicAdd(&p.heads[0], 1);
        // L2 hints: lines that will not be read again may go first; rows that may be read again
        // by the second pass get the default policy (0 = no hint).
        const uint64_t pol_keep = 0;
        const uint64_t pol_last_use = l2_policy_evict_first();
        const int P2 = p.plan.parts2;
        unsigned long long wait_t0 = 0;
        int cursor = 0;        // first published slot that may still have pieces
        bool again = false;    // the last look at the published slots found pieces left
        bool all_final = false;  // every sequence of the batch has been finalised
        int jb = -1, jn = 0, jpart = 0;  // final-token piece claimed for the next round
        bool piece_last = false;         // the previous round served a final-token piece
        while (ok) {
            // Published sequences form a global queue of (sequence, piece) served by every CTA in order:
            // each lane looks at one of the next 32 published slots; the first slot with pieces
            // left is tried with one atomic (an overshoot only means someone else was quicker).
            // A unit this CTA already holds a ticket for must not wait behind a long run of pieces
            // (its sequence could not finish): pieces and units alternate while both exist.
            jb = -1;
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
                cursor += done == 0xffffffffu ? 32 : __ffs(~done) - 1;    // skip leading exhausted slots
                again = open != 0;
                if (open) {
                    const int L = __ffs(open) - 1;
                    int piece = P2;
                    if (lane == L) piece = atomicAdd(&p.job_ctr[slot], 1);
                    piece = __shfl_sync(0xffffffffu, piece, L);
                    if (piece < P2) {
                        const unsigned long long el = __shfl_sync(0xffffffffu, e, L);
                        jb = (int)(el >> 32) - 1; jn = (int)(unsigned)el; jpart = piece;
                    }
                }
            }
            piece_last = jb >= 0;
            if (jb >= 0) {
                // 1. rows for a final token come first: they are hot in L2 right now
                __threadfence();
                const int b = jb, n = jn;          // n < K: the first rejected position
                const int step = CHUNK_ELEMS / 2;  // half a slot of each of the two rows
                const E* trow = tbase + (size_t)target_row(b, n, K) * V;
                const E* drow = dbase + (size_t)draft_row(b, n, K) * V;
                const float cj = PER_SEQ ? seq_c(p, b) : p.c;
                const int e_begin = jpart * p.plan.job_elems;
                const int e_end = min(V, e_begin + p.plan.job_elems);
                for (int e0 = e_begin; e0 < e_end; e0 += step, ++q) {
                    ok = loader_acquire(sm, q, lane);
                    if (!ok) break;
                    const int ne = min(step, e_end - e0);
                    const StageMeta mt{kFinal, b, ne, (e0 == e_begin ? 1 : 0) | (e0 + step >= e_end ? 2 : 0), e0, n, cj, 0};
                    loader_fill<E>(sm, q % STAGES, mt, use_tma, trow + e0, drow + e0, lane, pol_last_use);
                }
                if (!ok) break;
            } else if (!stats_done) {
                // 2. next piece of a row for the statistics pass
                if (sm.abort_flag) { ok = false; break; }
                const long long u = __shfl_sync(0xffffffffu, u_ahead, 0);
                if (u >= total_units) {
                    stats_done = true;   // nothing left to pull
                } else {
                    if (lane == 0) u_ahead = atomicAdd(&p.heads[0], 1);
                    const int b = (int)(u / (R * P));
                    const int rem = (int)(u % (R * P));
                    const int ridx = rem / P, part = rem % P;
                    const E* row = (ridx == 2 * K) ? tbase + (size_t)target_row(b, K, K) * V
                                                   : ((ridx & 1) ? dbase + (size_t)draft_row(b, ridx >> 1, K) * V
                                                                 : tbase + (size_t)target_row(b, ridx >> 1, K) * V);
                    const float cu = PER_SEQ ? seq_c(p, b) : p.c;
                    const int ch0 = part * cpp;
                    const int ch1 = min(chunks_per_row, ch0 + cpp);
                    for (int ch = ch0; ch < ch1; ++ch, ++q) {
                        ok = loader_acquire(sm, q, lane);
                        if (!ok) break;
                        const int e0 = ch * CHUNK_ELEMS;
                        const StageMeta mt{kStats, (int)u, min(CHUNK_ELEMS, V - e0), (ch == ch0 ? 1 : 0) | (ch == ch1 - 1 ? 2 : 0), e0, ridx == 2 * K ? 1 : 0, cu, 0};
                        // the extra target row is never streamed again (its sums are kept); the other
                        // rows may be, if their position turns out to be the first rejection
                        loader_fill<E>(sm, q % STAGES, mt, use_tma, row + e0, nullptr, lane, ridx == 2 * K ? pol_last_use : pol_keep);
                    }
                    if (!ok) break;
                }
            } else {
                // 3. No units left.  Stay and help with final-token pieces until every sequence of the
                //    batch has been finalised (by whichever CTA) and no piece is left to claim:
                //    leaving earlier would let the last sequences fall to very few CTAs.  The wait
                //    cannot deadlock: a sequence is finalised by CTAs that already hold its units,
                //    and those never wait for anyone.  It is bounded like every other wait.
                if (!again) {
                    if (all_final) break;   // seen before the look above, so that look was complete
                    int fin = 0;
                    if (lane == 0) {
                        fin = *reinterpret_cast<volatile int*>(&p.heads[1]) >= p.B ? 1 : 0;
                        if (!fin) {
                            if (sm.abort_flag) fin = -1;
                            const unsigned long long now = global_timer_ns();
                            if (wait_t0 == 0) wait_t0 = now;
                            else if (now - wait_t0 > kIdleLimitNs) { sm.abort_flag = 1; fin = -1; }
                            __nanosleep(50);
                        }
                    }
                    fin = __shfl_sync(0xffffffffu, fin, 0);
                    if (fin < 0) { ok = false; break; }
                    if (fin > 0) { all_final = true; __threadfence(); }
                }
            }
        }
        if (ok && loader_acquire(sm, q, lane)) {
            loader_fill<E>(sm, q % STAGES, StageMeta{kEnd, 0, 0, 0, 0, 0, 0.f, 0}, use_tma, (const E*)nullptr, (const E*)nullptr, lane, pol_keep);
        } else if (use_tma && lane == 0) {
            loader_drain(sm, q);
        }
    } else if (warp == kEpilogueWarp) {
        // =============================== epilogue warp
        // Takes up to 32 messages at a time.  Pieces are published in parallel (one lane each:
        // store, fence, ticket); what needs the whole warp then runs in message order.
        bool running = true;
        while (running) {
            int first = 0, cnt = 0;
            if (lane == 0) cnt = sm.epi.wait_batch(&first, &sm.abort_flag, kIdleLimitNs);
            cnt = __shfl_sync(0xffffffffu, cnt, 0);
            first = __shfl_sync(0xffffffffu, first, 0);
            if (cnt < 0) break;
            __threadfence_block();
            Msg m{kMsgNone, 0, 0, 0};
            if (lane < cnt) m = sm.epi.peek(first + lane);
            __syncwarp();
            if (lane == 0) sm.epi.release(first + cnt);
            int last_b = -1;
            // every piece message names a unit slot: wait until all eight consumer warps are through
            bool slot_ok = true;
            int top = -1;
            if (m.kind == kMsgJobPiece || m.kind == kMsgPiece) {
                slot_ok = mbar_wait(&sm.unit_bar[m.c % kUnitSlots], (m.c / kUnitSlots) & 1, &sm.abort_flag);
                top = m.c;
            }
            float pm = -INFINITY, ps = 0.f, pw = 0.f;
            if (m.kind == kMsgPiece && slot_ok) {
                const float cu = PER_SEQ ? seq_c(p, m.a / (R * P)) : p.c;
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float4 v = sm.scratch[m.c % kUnitSlots][w];
                    merge_ms(pm, ps, v.x, v.y, cu);
                }
                if (ENT) {   // sum e t of the piece, relative to the piece's maximum (known now)
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float4 v = sm.scratch[m.c % kUnitSlots][w];
                        pw += rebase_sum_w(v.x, v.y, v.z, pm, cu).y;
                    }
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) top = max(top, __shfl_xor_sync(0xffffffffu, top, off));
            __syncwarp();
            if (lane == 0 && top >= 0) { __threadfence_block(); sm.units_read = top + 1; }
            if (m.kind == kMsgJobPiece && slot_ok) {
                if (ticket_add(&p.ticket2[m.a]) == p.plan.parts2 - 1) last_b = m.a;  // all masses summed
            }
            if (m.kind == kMsgPiece && slot_ok) {
                const int b = m.a / (R * P);
                const int rem = m.a % (R * P);
                p.partial[((size_t)b * R + rem / P) * P + rem % P] = make_float2(pm, ps);
                if (ENT) p.partial_w[((size_t)b * R + rem / P) * P + rem % P] = pw;
                // two-level count (row, then sequence) spreads the atomics over many addresses
                bool row_done = true;
                if (P > 1) row_done = ticket_add(&p.ticket_row[(size_t)b * R + rem / P]) == P - 1;
                if (row_done && ticket_add(&p.ticket1[b]) == R - 1) last_b = b;  // last row of the sequence
            }
            // What needs a whole warp (decisions, final pick) goes to a global queue served by the
            // sequence warps of all CTAs: the CTA that happens to deliver the last piece of many
            // sequences (typically a slow one) must not also do all their epilogues.
            for (int i = 0; i < cnt && running; ++i) {
                const int kind = __shfl_sync(0xffffffffu, m.kind, i);
                const int a = __shfl_sync(0xffffffffu, m.a, i);
                const int bb = __shfl_sync(0xffffffffu, m.b, i);
                const int lb = __shfl_sync(0xffffffffu, last_b, i);
                if ((kind == kMsgPiece || kind == kMsgJobPiece) && lb >= 0 && lane == 0) {
                    const unsigned long long item = (1ull << 63) | ((unsigned long long)lb << 32) |
                                                    (kind == kMsgPiece ? 0xffffffffull : (unsigned long long)(unsigned)bb);
                    __threadfence();  // everything counted so far is visible before the item is
                    const int slot = atomicAdd(&p.heads[4], 1);
                    *reinterpret_cast<volatile unsigned long long*>(&p.wq[slot]) = item;
                }
                if (kind == kMsgExit) {
                    int pushed = 1;
                    if (lane == 0) pushed = sm.seq.push(Msg{kMsgExit, 0, 0, 0}, &sm.abort_flag, kWaitLimitNs) ? 1 : 0;
                    (void)__shfl_sync(0xffffffffu, pushed, 0);
                    running = false;
                }
            }
        }
    } else if (warp == kSequenceWarp) {
        // =============================== sequence warp: per-sequence decisions and the final pick
        // Serves the global queue of sequence work (any CTA's sequences).  Leaves when its own
        // CTA has wound down and nothing can be claimed: whatever a CTA's epilogue warp published
        // was published before that CTA's exit message, so the publisher's own sequence warp at
        // the latest picks it up.
        bool exiting = false;
        unsigned long long idle_t0 = 0;
        for (;;) {
            int kind = -1, b = 0, n = 0;   // kind 0: decide the sequence, 1: final pick after the second pass
            if (lane == 0) {
                Msg m{kMsgNone, 0, 0, 0};
                if (!exiting && sm.seq.try_pop(m) && m.kind == kMsgExit) kind = 2;
                if (kind < 0) {
                    for (int tries = 0; tries < 64; ++tries) {
                        const int h = *reinterpret_cast<volatile int*>(&p.heads[5]);
                        if (h >= 2 * p.B) break;
                        const unsigned long long e = *reinterpret_cast<volatile unsigned long long*>(&p.wq[h]);
                        if (e == 0) break;                               // nothing published there (yet)
                        if (atomicCAS(&p.heads[5], h, h + 1) == h) {
                            b = (int)((e >> 32) & 0x7fffffffu);
                            n = (int)(unsigned)e;
                            kind = (unsigned)e == 0xffffffffu ? 0 : 1;
                            break;
                        }
                    }
                }
                if (kind < 0 && sm.abort_flag) kind = 3;
            }
            kind = __shfl_sync(0xffffffffu, kind, 0);
            if (kind == 3) break;
            if (kind == 2) { exiting = true; continue; }
            if (kind < 0) {
                if (exiting) break;
                if (lane == 0) {
                    const unsigned long long now = global_timer_ns();
                    if (idle_t0 == 0) idle_t0 = now;
                    else if (now - idle_t0 > kIdleLimitNs) sm.abort_flag = 1;
                    __nanosleep(300);
                }
                continue;
            }
            b = __shfl_sync(0xffffffffu, b, 0);
            n = __shfl_sync(0xffffffffu, n, 0);
            idle_t0 = 0;
            __threadfence();
            if (kind == 0) {
                n = finalize_sequence<E, ENT>(p, b, lane);
                if (n == K) {
                    // every draft accepted: the sums of the extra row are already there
                    __threadfence();
                    __syncwarp();
                    select_token<E>(p, b, n, lane);
                } else if (n >= 0) {
                    // publish the sequence for the second pass; its row statistics first
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) {
                        const int slot = atomicAdd(&p.heads[3], 1);
                        *reinterpret_cast<volatile unsigned long long*>(&p.ready[slot]) =
                            ((unsigned long long)(b + 1) << 32) | (unsigned)n;
                    }
                }
                if (lane == 0) {  // finalised (valid or not): lets idle CTAs know when to leave
                    __threadfence();
                    atomicAdd(&p.heads[1], 1);
                }
            } else {
                select_token<E>(p, b, n, lane);
            }
        }
    } else {
        // =============================== consumer warps
        RowAccT<ENT> acc;
        acc_open(acc);
        int unit_ends = 0;   // ends of units and pieces seen so far (same in every consumer warp)
        RowNorm rn{0.f, 0.f, 0.f, 0.f, 0.0};
        for (uint32_t q = 0;; ++q) {
            const int stage = q % STAGES;
            if (!mbar_wait(&sm.full[stage], (q / STAGES) & 1u, &sm.abort_flag)) break;
            const StageMeta mt = sm.meta[stage];
            if (mt.kind == kEnd) {
                if (warp == 0 && lane == 0) sm.epi.push(Msg{kMsgExit, 0, 0, 0}, &sm.abort_flag, kWaitLimitNs);
                break;
            }
            if (mt.kind == kStats) {
                if (mt.flags & 1) acc_open(acc);
                if (mt.aux) {  // a piece of the extra target row
                    BonusSeg* out = bonus_segs(p, mt.id / (R * P)) + (size_t)(mt.elem0 / CHUNK_ELEMS) * kConsumerWarps + warp;
                    chunk_stats<E, true, ENT>(sm.buf[stage], mt.nelem, warp, lane, PER_SEQ ? mt.c : p.c, acc, out);
                } else {
                    chunk_stats<E, false, ENT>(sm.buf[stage], mt.nelem, warp, lane, PER_SEQ ? mt.c : p.c, acc, nullptr);
                }
                if (!(mt.flags & 2)) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.empty[stage]);
                    continue;
                }
                // last chunk of the unit: (max, sum) of the warp -- the maximum first (shuffles only),
                // then one rescale per thread and a sum
                const float cu = PER_SEQ ? mt.c : p.c;
                float wv = 0.f;
                const float2 ms = acc_close(acc, cu, &wv);
                float m = ms.x;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                const float2 sw = ENT ? rebase_sum_w(ms.x, ms.y, wv, m, cu) : make_float2(rebase_sum(ms.x, ms.y, m, cu), 0.f);
                float sum = sw.x, wsum = sw.y;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    sum += __shfl_xor_sync(0xffffffffu, sum, off);
                    if (ENT) wsum += __shfl_xor_sync(0xffffffffu, wsum, off);
                }
                if (lane == 0) {
                    const int us = unit_ends % kUnitSlots;
                    sm.scratch[us][warp] = make_float4(m, sum, wsum, 0.f);
                    mbar_arrive(&sm.unit_bar[us]);
                    if (warp == 0) push_unit_end(sm, Msg{kMsgPiece, mt.id, 0, unit_ends});
                    mbar_arrive(&sm.empty[stage]);
                }
                ++unit_ends;
                continue;
            }
            // the two rows of a rejected position: segment sums of max(0, P_t - P_d)
            const int b = mt.id, n = mt.aux;
            if (mt.flags & 1) {
                const float2 st = __ldcg(&p.rowstat[(size_t)b * R + 2 * n]);
                const float2 sd = __ldcg(&p.rowstat[(size_t)b * R + 2 * n + 1]);
                rn = make_rownorm(st, sd);
            }
            double* seg_out = seg_sums(p, b) + mt.elem0 / kSegElems;
            chunk_segments<E, true>(sm.buf[stage], sm.buf[stage] + kChunkBytes / 2, mt.nelem, warp, lane, rn, PER_SEQ ? mt.c : p.c, seg_out);
            if (mt.flags & 2) {
                // last chunk of the piece: publish the sums; the epilogue warp counts the piece once
                // all warps are through and, when it is the sequence's last, picks the token
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    mbar_arrive(&sm.unit_bar[unit_ends % kUnitSlots]);
                    if (warp == 0) push_unit_end(sm, Msg{kMsgJobPiece, b, n, unit_ends});
                }
                ++unit_ends;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
        }
    }
    if (sm.abort_flag && lane == 0) atomicOr(&p.heads[2], kDevTimeout);
}

}  // namespace ears
