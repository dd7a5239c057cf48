// C ABI of the EARS verification step (see include/ears.h): argument checks,
// launch plan, workspace management and the kernel launch.
#include "../../include/ears.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <type_traits>
#include <utility>
#include <vector>

#include "ears_common.cuh"
#include "ears_kernel.cuh"
#include "ears_resident.cuh"
#include "ears_greedy.cuh"
#include "ears_direct.cuh"
#include "ears_shard.cuh"
#include "ears_cstream.cuh"

namespace {

using namespace ears;

bool dtype_ok(int dtype) { return dtype == EARS_DTYPE_F32 || dtype == EARS_DTYPE_BF16 || dtype == EARS_DTYPE_F16; }
int dtype_size(int dtype) { return dtype == EARS_DTYPE_F32 ? 4 : 2; }

// Calls f with a null pointer to the element type of `dtype` (float, uint16_t = bfloat16 bits, f16_t).
template <typename F>
int by_dtype(int dtype, F&& f) {
    if (dtype == EARS_DTYPE_F32) return f((float*)nullptr);
    if (dtype == EARS_DTYPE_F16) return f((f16_t*)nullptr);
    return f((uint16_t*)nullptr);
}

// 256 KB of one row per unit when there is plenty of work (smaller units cost more per-unit
// bookkeeping than they gain in balance; measured on B=512, V=256000).
constexpr int kUnitChunks = 16;

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", what, cudaGetErrorString(e));
    return EARS_ERR_CUDA;
}
#define EARS_CUDA(call)                                     \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

struct PlanOverride { int loader = 0, parts1 = 0, path = 0, cluster = 0; };

// Initial choice of kernel from the environment (EARS_PATH=streaming|resident|direct, EARS_CLUSTER=1..16),
// for trying a launch plan on an unmodified caller; ears_set_path overrides it.
PlanOverride override_from_env() {
    PlanOverride ov;
    if (const char* e = getenv("EARS_PATH")) {
        if (!strcmp(e, "streaming") || !strcmp(e, "1")) ov.path = 1;
        else if (!strcmp(e, "resident") || !strcmp(e, "2")) ov.path = 2;
        else if (!strcmp(e, "direct") || !strcmp(e, "3")) ov.path = 3;
        else if (!strcmp(e, "cluster-streamed") || !strcmp(e, "4")) ov.path = 4;
    }
    if (const char* e = getenv("EARS_CLUSTER")) {
        const int c = atoi(e);
        if (c == 1 || c == 2 || c == 4 || c == 8 || c == 16) ov.cluster = c;
    }
    return ov;
}
PlanOverride g_override = override_from_env();
std::mutex g_mutex;

struct DeviceInfo {
    int sms = 0;
    bool attrs_set = false;
    bool cluster16 = false;                        // clusters of 16 CTAs may be launched
    std::map<std::pair<int, int>, int> clusters;   // (cluster size, shared memory, element size) -> co-resident clusters
};
std::map<int, DeviceInfo> g_devices;

struct Buffer {
    void* ptr = nullptr;
    size_t bytes = 0;
    // Library-owned workspaces carry two copies of the counter block.  A call uses one and its
    // kernel zeroes the other for the next call of the same shape, which then needs no memset
    // (and starts clean even if this call was cut short by a device-side timeout).
    int clean_set = -1;            // copy that is known to be all zero, -1: none
    unsigned long long sig = 0;    // kernel kind and sizes the copies were laid out for
    void* status_word = nullptr;   // status word of the most recent call
    bool captured = false;         // a call on this workspace was recorded into a CUDA graph: its replays use
                                   // copy 0 behind the host's back, so from then on every call clears copy 0 itself
};
std::map<std::pair<int, void*>, Buffer> g_workspaces;  // (device, stream) -> scratch
std::map<std::pair<int, void*>, Buffer> g_staging;     // (device, stream) -> host-entry staging
// Workspaces that a CUDA graph may still point at: kept until ears_shutdown (device, pointer).
std::vector<std::pair<int, void*>> g_parked;

struct Profile {
    bool active = false;
    int max_calls = 0;
    size_t used = 0;                  // events recorded so far
    std::vector<cudaEvent_t> events;  // 2 per timed call, created by ears_profile_begin
} g_profile;

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// pieces per row and chunks per piece for `items` rows of `chunks` chunks each
void split_rows(long long items, int chunks, int sms, int forced_parts, int* parts, int* cpp) {
    int c = kUnitChunks;
    const long long want_units = 8LL * sms;
    if (items * ((chunks + c - 1) / c) < want_units) {
        long long per_row = (want_units + items - 1) / items;  // desired pieces per row
        if (per_row > chunks) per_row = chunks;
        c = (int)(chunks / per_row);
        if (c < 1) c = 1;
    }
    if (forced_parts > 0) {
        int fp = forced_parts > chunks ? chunks : forced_parts;
        c = (chunks + fp - 1) / fp;
    }
    if (c > chunks) c = chunks;
    // equal pieces: 19 chunks in 2 pieces are 10 + 9, not 16 + 3
    const int n = (chunks + c - 1) / c;
    c = (chunks + n - 1) / n;
    *cpp = c;
    *parts = (chunks + c - 1) / c;
}

// Which of the two streaming kernels takes a shape the resident kernel does not.  The kernel that
// reads straight from global memory wins on 2-byte logits (its warps do not march in step, which
// the special-function pipe rewards) and on short rows (no per-slot costs), from a few hundred
// positions on; the ring kernel keeps long 4-byte rows (HBM-bound either way) and small batches
// (shorter tail).  Measured on B200, us direct / ring: 1024,4,152064,bf16: 562 / 734;
// 128,4,152064,bf16: 120 / 144; 64,4,152064,bf16: 100 / 94; 2048,4,32000,fp32: 485 / 1200;
// 512,3,256000,fp32: 592 / 571.
bool use_direct(const PlanOverride& ov, int esize, int V, long long items) {
    if (ov.path == 1) return false;
    if (ov.path == 3) return true;
    if (ov.parts1 != 0) return false;               // the piece count is a knob of the ring kernel's tests
    if (items < 400) return false;
    return esize == 2 || (long long)V * esize <= 512 * 1024;
}

Plan make_plan(int B, int K, int V, int esize, bool aligned, int sms, const PlanOverride& ov, bool direct = false) {
    Plan pl;
    const int chunk_elems = kChunkBytes / esize;
    const int chunks = (V + chunk_elems - 1) / chunk_elems;
    pl.use_tma = aligned && ov.loader != 2;
    split_rows((long long)B * (2 * K + 1), chunks, sms, ov.parts1, &pl.parts1, &pl.cpp1);
    if (direct && ov.parts1 == 0 && pl.cpp1 < 4) {
        // the kernel that reads straight from global memory keeps eight 16-byte loads per thread
        // in flight: pieces below 64 KB would leave most of that unused
        const int n = (chunks + 3) / 4;
        pl.cpp1 = (chunks + n - 1) / n;
        pl.parts1 = (chunks + pl.cpp1 - 1) / pl.cpp1;
    }
    pl.nseg = (V + kSegElems - 1) / kSegElems;
    const long long ctas = (long long)sms * kCtasPerSm;
    // second pass (rejected positions): 64 KB of each row per piece, single chunks when there are few sequences
    int job_chunks = (long long)B * ((chunks + 3) / 4) >= ctas ? 4 : 1;
    if (direct && job_chunks < 2 && esize == 4) job_chunks = 2;   // a round of its second pass covers 8192 entries
    pl.job_elems = job_chunks * chunk_elems;
    pl.parts2 = (V + pl.job_elems - 1) / pl.job_elems;
    return pl;
}

struct Layout {
    size_t ticket1, ticket2, job_ctr, ticket_row, ready, heads, wq, counters_bytes;
    size_t partial, rowstat, partial_w, roww, pt_tok, pd_tok, max_pt, cls, resid, seg, seg_stride, total;
};

Layout make_layout(int B, int K, int V, int parts1) {
    Layout L;
    const size_t rows = (size_t)B * (2 * K + 1);
    size_t o = 0;
    L.heads = o; o += kHeadsWords * 4;  // fixed place: the status word is heads[2] of any workspace, the decision counts heads[8..11]
    L.wq = o; o += (size_t)B * 16;
    L.ticket1 = o; o += (size_t)B * 4;
    L.ticket2 = o; o += (size_t)B * 4;
    L.job_ctr = o; o += (size_t)B * 4;
    L.ticket_row = o; o += rows * 4;
    o = align_up(o, 8);
    L.ready = o; o += (size_t)B * 8;
    L.counters_bytes = o;
    o = align_up(o, 256);
    L.partial = o; o = align_up(o + rows * parts1 * sizeof(float2), 256);
    L.rowstat = o; o = align_up(o + rows * sizeof(float2), 256);
    L.partial_w = o; o = align_up(o + rows * parts1 * sizeof(float), 256);   // (entropy kernels)
    L.roww = o; o = align_up(o + rows * sizeof(float), 256);
    L.pt_tok = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.pd_tok = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.max_pt = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.cls = o; o = align_up(o + (size_t)B * K, 256);
    L.resid = o; o = align_up(o + (size_t)B * 8, 256);
    // per sequence: BonusSeg per (chunk, consumer warp) of the extra row, later reused for the
    // second pass's segment sums; 4-byte elements give the most chunks
    const size_t bonus_bytes = (size_t)((V + kChunkBytes / 4 - 1) / (kChunkBytes / 4)) * kConsumerWarps * sizeof(BonusSeg);
    const size_t seg_bytes = (size_t)((V + kSegElems - 1) / kSegElems) * sizeof(double);
    L.seg_stride = align_up(bonus_bytes > seg_bytes ? bonus_bytes : seg_bytes, 16);
    L.seg = o; o = align_up(o + (size_t)B * L.seg_stride, 256);
    L.total = o;
    return L;
}

// ---- the resident path: one position's rows held in the shared memory of a cluster ----
struct RPlan {
    bool ok = false;
    int C = 0, slice = 0, buf_bytes = 0;
    size_t smem = 0;
    bool roomy = false, streamed = false;
    int job_elems = 0, parts2 = 0;   // streaming clusters: entries per second-pass piece, pieces per job
};

size_t resident_smem(int buf_bytes) { return ((sizeof(RSmem) + 127) & ~size_t(127)) + 2 * (size_t)buf_bytes + 128; }

// Three CTAs per SM (74 KB each) when the slices allow it, else two (113 KB each); a pair of
// rows that does not fit a cluster that way goes to the streaming kernel.
constexpr size_t kResidentSmem3 = 74 * 1024, kResidentSmem2 = 113 * 1024;

RPlan make_rplan(int B, int K, int V, int esize, int sms, int max_cluster, int forced_cluster) {
    RPlan best;
    const long long items = (long long)B * (K + 1);
    for (int pass = 0; pass < 2 && !best.ok; ++pass) {
        const size_t cap = pass == 0 ? kResidentSmem3 : kResidentSmem2;
        for (int C = 1; C <= max_cluster; C *= 2) {
            if (forced_cluster > 0 && C != forced_cluster) continue;
            const int slice = (int)align_up((size_t)((V + C - 1) / C), kSegElems);
            const int buf = (int)align_up((size_t)slice * esize, kRSubBytes);
            if (buf > kRMaxSub * kRSubBytes || resident_smem(buf) > cap) continue;
            if (best.ok && items * best.C >= 2LL * sms) break;   // enough CTAs already: keep the slices large
            best.ok = true; best.C = C; best.slice = slice; best.buf_bytes = buf; best.smem = resident_smem(buf);
            best.roomy = pass == 0;
        }
    }
    return best;
}

// The streamed form of the cluster kernel: nothing is staged, a CTA only keeps the extra row's
// sums per 2 KB of its slice.  Cluster size: a CTA pulls some 20 GB/s on its own, so positions are
// split over as many CTAs as it takes to fill the CTA slots of the device in one round, and no
// further -- a second, mostly empty round costs more than longer slices do (measured on B200, us for
// clusters of 1 / 2 / 4: 32 x 8 positions of 2 x 256 KB: 60 / 73 / 79; 64 x 8: 95 / 97 / 119;
// 128 x 5 of 2 x 304 KB: 111 / 115 / 145; 32 x 4 of 2 x 1 MB (4-byte): 97 / 72 / 86).  When sequences
// are walked in order a small model of the launch picks the size instead: rounds x positions in a row
// x (time to stream a position + its exchange, decision and report).
constexpr size_t kStreamedSegBytes = 48 * 1024;   // segment sums of a slice: at most this much shared memory

// bytes behind CSmem: the extra row's sums per 2 KB of the slice (sized for 4-byte entries, which give the most)
size_t streamed_area(int slice) {
    return ((size_t)slice * 4 / kBonusSegBytes + kCBonusPad) * sizeof(BonusSeg);
}
// behind the sums, 128-byte aligned: the copy ring
size_t streamed_ring_offset(int slice) { return align_up(streamed_area(slice), 128); }
size_t streamed_smem(int slice, int esize) {   // (only 4-byte logits use the ring)
    return ((sizeof(CSmem) + 127) & ~size_t(127)) + streamed_ring_offset(slice) + (esize == 4 ? (size_t)kCStages * kCStageBytes : 0) + 128;
}

RPlan make_splan(int B, int K, int V, int esize, int sms, int max_cluster, int forced_cluster, bool ordered) {
    RPlan best;
    double best_t = 0.0;
    const long long items = ordered ? (long long)B : (long long)B * (K + 1);
    const double item_bytes = 2.0 * V * esize;
    for (int C = 1; C <= max_cluster; C *= 2) {
        if (forced_cluster > 0 && C != forced_cluster) continue;
        const int slice = (int)align_up((size_t)((V + C - 1) / C), kCSliceAlign);
        if (streamed_area(slice) > kStreamedSegBytes) continue;
        const long long resident = std::max<long long>(1, (long long)kCCtasPerSm * sms / C);
        const long long clusters = std::min(items, resident);
        const long long rounds = (items + clusters - 1) / clusters;
        // per position: its bytes at the share of ~6.5 TB/s that the active CTAs leave it, but no faster than
        // one CTA can pull on its own (~60 GB/s), plus ~2.5 us of exchange, decision and report
        const double share = 6.5e12 / (double)(clusters * C);
        const double t_item = item_bytes / C / std::min(share, 60e9) + 2.5e-6;
        double t = rounds * t_item * (K + 1);   // walking a sequence in order: up to K+1 positions in a row
        if (!ordered) t = items <= resident ? -(double)C : (double)C;   // the largest size whose clusters all run in one round, else the smallest
        if (!best.ok || t < best_t) {
            best.ok = true; best.C = C; best.slice = slice; best.buf_bytes = (int)streamed_ring_offset(slice); best.smem = streamed_smem(slice, esize);
            best.roomy = true; best.streamed = true;
            best_t = t;
        }
    }
    if (best.ok) {
        // Pieces of a job (a sequence's first rejected position) in the shared queue: 16 KB of each row
        // (32 KB for 4-byte entries: one sweep of a CTA's warps), so that the many CTAs waiting at the end
        // of a small batch finish a job in one short step.
        const int chunk_elems = kChunkBytes / esize;
        // (twice that once the positions give every CTA four rounds or more: CTAs are busy then, and the
        // round trips around a piece weigh more than the wait for a job's last piece)
        const int job_chunks = (esize == 4 ? 2 : 1) * (items >= 4LL * kCCtasPerSm * sms ? 2 : 1);
        best.job_elems = job_chunks * chunk_elems;
        best.parts2 = (V + best.job_elems - 1) / best.job_elems;
    }
    return best;
}

struct RLayout {
    size_t heads, ticket, ticket2, seqmask, ready, counters_bytes, flag, cand, cand_mass, rowstat, pt_tok, pd_tok, max_pt, cls, resid,
        seg, total;
    int nseg;
};

RLayout make_rlayout(int B, int K, int V) {
    RLayout L;
    size_t o = 0;
    L.heads = o; o += kHeadsWords * 4;   // the status word is heads[2] of any workspace
    L.ticket = o; o += (size_t)B * 4;
    L.ticket2 = o; o += (size_t)B * 4;
    o = align_up(o, 8);
    L.seqmask = o; o += (size_t)B * 8;
    L.ready = o; o += (size_t)B * 8;
    L.counters_bytes = o;
    o = align_up(o, 256);
    L.flag = o; o = align_up(o + (size_t)B * (K + 1), 256);
    L.cand = o; o = align_up(o + (size_t)B * (K + 1) * 4, 256);
    L.cand_mass = o; o = align_up(o + (size_t)B * (K + 1) * 8, 256);
    L.rowstat = o; o = align_up(o + (size_t)B * (K + 1) * 16, 256);
    L.pt_tok = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.pd_tok = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.max_pt = o; o = align_up(o + (size_t)B * K * 8, 256);
    L.cls = o; o = align_up(o + (size_t)B * K, 256);
    L.resid = o; o = align_up(o + (size_t)B * 8, 256);
    L.nseg = (V + kSegElems - 1) / kSegElems;   // (streaming clusters: the second pass's sums per segment)
    L.seg = o; o = align_up(o + (size_t)B * L.nseg * 8, 256);
    L.total = o;
    return L;
}

// ---- the greedy (temperature -> 0) form ----
struct GLayout { size_t heads, ticket, counters_bytes, partial, total; int P, piece_elems; };

GLayout make_glayout(int B, int K, int V, int esize, int sms) {
    GLayout L;
    const long long rows = (long long)B * (K + 1);
    // pieces of at least 16 KB, enough of them to give every CTA several
    const long long row_bytes = (long long)V * esize;
    long long maxp = row_bytes / 16384;
    if (maxp < 1) maxp = 1;
    long long want = (8LL * sms + rows - 1) / rows;
    if (want < 1) want = 1;
    long long P = want < maxp ? want : maxp;
    if (P > 4096) P = 4096;
    long long pe = (V + P - 1) / P;
    pe = (long long)align_up((size_t)pe, kSegElems);
    L.piece_elems = (int)pe;
    L.P = (int)((V + pe - 1) / pe);
    size_t o = 0;
    L.heads = o; o += kHeadsWords * 4;
    L.ticket = o; o += (size_t)B * 4;
    L.counters_bytes = o;
    o = align_up(o, 256);
    L.partial = o; o = align_up(o + (size_t)rows * L.P * sizeof(int4), 256);
    L.total = o;
    return L;
}

int check_shape(int B, int K, int V) {
    if (B < 1 || K < 1 || V < 1) return EARS_ERR_SHAPE;
    if (K > EARS_MAX_K || V > (1 << 30)) return EARS_ERR_SHAPE;
    // element and unit counts must stay far inside 63 / 31 bits
    const long double elems = (long double)B * (K + 1) * V;
    if (elems * 4 > 4.0e18L) return EARS_ERR_SHAPE;
    if ((long double)B * (2 * K + 1) * 64 > 2.0e9L) return EARS_ERR_SHAPE;
    return EARS_OK;
}

int device_info(int dev, DeviceInfo** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& di = g_devices[dev];
    if (di.sms == 0) {
        int sms = 0;
        EARS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        di.sms = sms;
    }
    *out = &di;
    return EARS_OK;
}

size_t smem_bytes() { return sizeof(PipeSmem<kStages>) + 128; }

// The events exist already (ears_profile_begin): a timed call only records them.
bool profile_wanted() { return g_profile.active && g_profile.used + 2 <= g_profile.events.size(); }

int profile_mark(cudaStream_t stream, bool timed) {
    if (!timed) return EARS_OK;
    EARS_CUDA(cudaEventRecord(g_profile.events[g_profile.used++], stream));
    return EARS_OK;
}

template <typename E>
int set_attrs_streamed(bool* cluster16) {
    EARS_CUDA(cudaFuncSetAttribute(ears_cstream_kernel<E, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)(streamed_smem(0, (int)sizeof(E)) + kStreamedSegBytes)));
    EARS_CUDA(cudaFuncSetAttribute(ears_cstream_kernel<E, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)(streamed_smem(0, (int)sizeof(E)) + kStreamedSegBytes)));
    if (cudaFuncSetAttribute(ears_cstream_kernel<E, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(ears_cstream_kernel<E, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        (void)cudaGetLastError();
        *cluster16 = false;
    }
    return EARS_OK;
}

template <typename E>
int set_attrs(bool* cluster16) {
    int rc = set_attrs_streamed<E>(cluster16);
    if (rc) return rc;
    EARS_CUDA(cudaFuncSetAttribute(ears_verify_kernel<E, kStages, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes()));
    EARS_CUDA(cudaFuncSetAttribute(ears_verify_kernel<E, kStages, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes()));
    EARS_CUDA(cudaFuncSetAttribute(ears_verify_kernel<E, kStages, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes()));
    EARS_CUDA(cudaFuncSetAttribute(ears_verify_kernel<E, kStages, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes()));
    EARS_CUDA(cudaFuncSetAttribute(ears_resident_kernel<E, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kResidentSmem2));
    EARS_CUDA(cudaFuncSetAttribute(ears_resident_kernel<E, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kResidentSmem2));
    // several CTAs per SM only fit when the SM's memory is configured as shared memory
    EARS_CUDA(cudaFuncSetAttribute(ears_resident_kernel<E, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   (int)cudaSharedmemCarveoutMaxShared));
    EARS_CUDA(cudaFuncSetAttribute(ears_resident_kernel<E, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   (int)cudaSharedmemCarveoutMaxShared));
    // clusters of more than 8 CTAs are an opt-in; without it the plans stop at 8
    if (cudaFuncSetAttribute(ears_resident_kernel<E, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
        cudaFuncSetAttribute(ears_resident_kernel<E, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        (void)cudaGetLastError();
        *cluster16 = false;
    }
    return EARS_OK;
}

// How many clusters of this shape the device can hold at once (cached per device).
template <typename E>
int resident_clusters(DeviceInfo* di, const RPlan& rp, int dtype, int* out) {
    const std::pair<int, int> key(rp.C * 16 + dtype * 2 + (rp.streamed ? 1 : 0), (int)rp.smem);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        auto it = di->clusters.find(key);
        if (it != di->clusters.end()) { *out = it->second; return EARS_OK; }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(rp.C * di->sms), 1, 1);
    cfg.blockDim = dim3(rp.streamed ? kCThreads : kRThreads, 1, 1);
    cfg.dynamicSmemBytes = rp.smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)rp.C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    // (the entropy variants have the same footprint)
    const cudaError_t qe = rp.streamed ? cudaOccupancyMaxActiveClusters(&n, ears_cstream_kernel<E, false>, &cfg)
                                       : cudaOccupancyMaxActiveClusters(&n, ears_resident_kernel<E, false>, &cfg);
    if (qe != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    di->clusters[key] = n;
    *out = n;
    return EARS_OK;
}

template <typename E>
int launch_resident(RParams& p, const RPlan& rp, int max_clusters, cudaStream_t stream) {
    const long long items = p.ordered ? (long long)p.B : (long long)p.B * (p.K + 1);
    p.n_clusters = (int)(items < max_clusters ? items : max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.n_clusters * rp.C), 1, 1);
    cfg.blockDim = dim3(rp.streamed ? kCThreads : kRThreads, 1, 1);
    cfg.dynamicSmemBytes = rp.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)rp.C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool timed = profile_wanted();
    int rc = profile_mark(stream, timed);
    if (rc) return rc;
    const bool ent = p.unc_entropy || p.entropy;
    if (rp.streamed && ent) EARS_CUDA(cudaLaunchKernelEx(&cfg, ears_cstream_kernel<E, true>, p));
    else if (rp.streamed) EARS_CUDA(cudaLaunchKernelEx(&cfg, ears_cstream_kernel<E, false>, p));
    else if (ent) EARS_CUDA(cudaLaunchKernelEx(&cfg, ears_resident_kernel<E, true>, p));
    else EARS_CUDA(cudaLaunchKernelEx(&cfg, ears_resident_kernel<E, false>, p));
    return profile_mark(stream, timed);
}

template <typename E>
int launch(const Params& p, int sms, bool direct, cudaStream_t stream) {
    const long long units = (long long)p.B * (2 * p.K + 1) * p.plan.parts1;
    const long long cap = (long long)sms * kCtasPerSm;
    const int grid = (int)(units < cap ? units : cap);
    const bool timed = profile_wanted();
    int rc = profile_mark(stream, timed);
    if (rc) return rc;
    const bool ent = p.unc_entropy || p.entropy;
    if (direct) {
        const long long dcap = (long long)sms * kDCtasPerSm;
        const int dgrid = (int)(units < dcap ? units : dcap);
        if (p.seq_T && ent) ears_direct_kernel<E, true, true><<<dgrid, kDThreads + 32, 0, stream>>>(p);
        else if (p.seq_T) ears_direct_kernel<E, true, false><<<dgrid, kDThreads + 32, 0, stream>>>(p);
        else if (ent) ears_direct_kernel<E, false, true><<<dgrid, kDThreads + 32, 0, stream>>>(p);
        else ears_direct_kernel<E, false, false><<<dgrid, kDThreads + 32, 0, stream>>>(p);
    } else if (p.seq_T && ent) {
        ears_verify_kernel<E, kStages, true, true><<<grid, kThreads, smem_bytes(), stream>>>(p);
    } else if (p.seq_T) {
        ears_verify_kernel<E, kStages, true, false><<<grid, kThreads, smem_bytes(), stream>>>(p);
    } else if (ent) {
        ears_verify_kernel<E, kStages, false, true><<<grid, kThreads, smem_bytes(), stream>>>(p);
    } else {
        ears_verify_kernel<E, kStages, false, false><<<grid, kThreads, smem_bytes(), stream>>>(p);
    }
    EARS_CUDA(cudaGetLastError());
    return profile_mark(stream, timed);
}

int get_buffer(std::map<std::pair<int, void*>, Buffer>& pool, int dev, void* stream, size_t bytes, void** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    Buffer& b = pool[std::make_pair(dev, stream)];
    if (b.bytes < bytes) {
        if (b.ptr && b.captured) {
            // A call on this buffer was recorded into a CUDA graph whose replays will use these very
            // addresses: the buffer is never freed before ears_shutdown.  Later eager calls move to
            // a new one (replays and eager calls stay ordered by the stream they share).
            g_parked.emplace_back(dev, b.ptr);
            b.ptr = nullptr;
            b.bytes = 0;
            b.captured = false;
        } else if (b.ptr) {
            // work enqueued earlier on this stream may still use the old buffer
            EARS_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
            EARS_CUDA(cudaFree(b.ptr));
            b.ptr = nullptr;
            b.bytes = 0;
        }
        const size_t want = align_up(bytes + bytes / 4, 1 << 20);
        EARS_CUDA(cudaMalloc(&b.ptr, want));
        b.bytes = want;
        b.clean_set = -1;
        b.status_word = nullptr;
    }
    *out = b.ptr;
    return EARS_OK;
}

// A launch that failed has not cleared the other copy: the next call must start with a memset.
void forget_clean_counters(int dev, void* stream_) {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_workspaces.find(std::make_pair(dev, stream_));
    if (it != g_workspaces.end()) it->second.clean_set = -1;
}

// Picks the counter block of a call on `stream`.  Caller-owned workspace: the block at its start,
// cleared by a memset.  Library-owned: see Buffer.  *zero_ptr / *zero_words name the other copy,
// which the kernel clears (0 words: nothing to clear).
int pick_counters(void* caller_ws, int dev, void* stream_, int kind, size_t counters_bytes, size_t total,
                  char** base, char** counters, int** zero_ptr, int* zero_words) {
    cudaStream_t stream = (cudaStream_t)stream_;
    const size_t cb = align_up(counters_bytes, 256);
    if (caller_ws) {
        *base = (char*)caller_ws;
        *counters = *base;
        *zero_ptr = nullptr;
        *zero_words = 0;
        EARS_CUDA(cudaMemsetAsync(*counters, 0, counters_bytes, stream));
        return EARS_OK;
    }
    void* ws = nullptr;
    const size_t main_bytes = align_up(total, 256);
    int rc = get_buffer(g_workspaces, dev, stream_, main_bytes + cb, &ws);
    if (rc) return rc;
    std::lock_guard<std::mutex> lock(g_mutex);
    Buffer& b = g_workspaces[std::make_pair(dev, stream_)];
    char* set[2] = {(char*)ws, (char*)ws + main_bytes};
    const unsigned long long sig = ((unsigned long long)kind << 60) ^ ((unsigned long long)counters_bytes << 32) ^ (unsigned long long)total;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    EARS_CUDA(cudaStreamIsCapturing(stream, &capturing));
    if (capturing != cudaStreamCaptureStatusNone) b.captured = true;
    int use = b.captured ? -1 : b.clean_set;
    if (use < 0 || b.sig != sig) {
        use = 0;
        EARS_CUDA(cudaMemsetAsync(set[0], 0, counters_bytes, stream));
    }
    b.sig = sig;
    b.clean_set = b.captured ? -1 : 1 - use;   // the kernel of this call clears the other copy
    b.status_word = set[use] + 2 * sizeof(int);
    *base = (char*)ws;
    *counters = set[use];
    *zero_ptr = (int*)set[1 - use];
    *zero_words = (int)(cb / sizeof(int));
    return EARS_OK;
}

// The cluster plan for this shape (rows resident in shared memory, or streamed by the clusters), if
// one of the two is the kernel to take.
int choose_resident(int dtype, int B, int K, int V, bool ordered, DeviceInfo* di, const PlanOverride& ov, RPlan* rp,
                    int* max_clusters) {
    *rp = RPlan();
    *max_clusters = 0;
    if (ov.path == 1 || ov.path == 3 || ov.parts1 != 0) return EARS_OK;
    const int esize = dtype_size(dtype);
    const int cmax = di->cluster16 ? kRMaxCluster : 8;
    const long long items = (long long)B * (K + 1);
    const long long slots = (long long)kCCtasPerSm * di->sms;
    auto clusters_of = [&](const RPlan& plan, int* out) {
        return by_dtype(dtype, [&](auto* e) { return resident_clusters<std::remove_pointer_t<decltype(e)>>(di, plan, dtype, out); });
    };
    if (ov.path == 4) {
        *rp = make_splan(B, K, V, esize, di->sms, cmax, ov.cluster, ordered);
    } else {
        *rp = make_rplan(B, K, V, esize, di->sms, cmax, ov.cluster);
        if (rp->ok) {
            const int rc = clusters_of(*rp, max_clusters);
            if (rc) return rc;
            if (*max_clusters < 1) rp->ok = false;
        }
    }
    if (ov.path == 0) {
        // Holding rows in shared memory costs a cluster about 6.5 us per position when it starts fresh and
        // 13 us in steady state, which nothing else in its CTAs can hide.  It wins when rows are short (a
        // cluster of at most four CTAs holds a pair: many clusters fit the device) and, with larger
        // clusters, while the positions take the resident clusters no more than two to three rounds.
        // Measured on B200 (B, K, V, dtype: us resident / cluster-streamed / best of ring and direct):
        // 8,5,32000,bf16: 19 / 25 / 38;  512,5,32000,bf16: 155 / 166 / 153;  4096,5,32000,bf16: 1048 / 1024 / 832;
        // 8,7,128256,bf16: 41 / 45 / 53;  16,7,128256,bf16: 49 / 49 / 61;  24,7,128256,bf16: 66 / 51 / 70;
        // 32,7,128256,bf16: 77 / 60 / 75;  8,4,152064,bf16: 37 / 45 / 50;  16,4,152064,bf16: 55 / 48 / 59.
        bool resident = rp->ok;
        if (resident) {
            const long long limit = !rp->roomy ? 64 : (rp->C >= 8 ? std::min<long long>(256, 8LL * *max_clusters / 3) : 3072);
            resident = items <= limit;
        }
        if (!resident) {
            // Clusters that stream their slices.  Their sweep is the fastest there is on 2-byte logits, and
            // a batch that gives the device's CTA slots only a few rounds of positions has the shortest tail
            // with them (the second pass of a first rejection is shared out piece by piece among all CTAs);
            // the streaming kernels' finer units win in larger batches, the ring kernel on long 4-byte rows
            // once the positions outnumber what two CTAs per SM take in one round.  Measured on B200 (B, K, V, dtype: us cluster-streamed /
            // best of ring and direct): 64,7,128256,bf16: 96 / 105;  128,..: 143 / 143;  160,..: 160 / 168;
            // 256,..: 225 / 229;  512,..: 428 / 399;  32,4,152064,bf16: 55 / 68;  64,..: 72 / 94;  128,..: 113 / 125;
            // 256,..: 164 / 186;  320,..: 209 / 220;  384,..: 239 / 246;  512,..: 295 / 309;  1024,..: 541 / 551 (643 / 621 at beta = 0);
            // 8,3,256000,fp32: 35 / 57;  32,..: 72 / 90;  64,..: 119 / 129;  96,..: 221 / 161;  128,..: 213 / 192.
            // With the flag that leaves out what follows a first rejection they also skip the reads, which
            // pays from four sequences per SM on.
            // (With the flag these clusters always walk sequences in order, a chain of up to K+1 positions
            // that a small batch cannot hide: below that size a flagged call goes to the streaming kernels.)
            const bool few = !ordered && (esize == 2 ? items <= 6 * slots : items <= 2LL * di->sms);
            const bool skip_reads = ordered && B >= 4 * di->sms;
            RPlan sp;
            if (few || skip_reads) sp = make_splan(B, K, V, esize, di->sms, cmax, ov.cluster, ordered);
            *rp = sp;   // (not ok: a streaming kernel takes the call)
            *max_clusters = 0;
        }
    }
    if (rp->ok && *max_clusters == 0) {
        const int rc = clusters_of(*rp, max_clusters);
        if (rc) return rc;
        if (*max_clusters < 1) rp->ok = false;
    }
    if (!rp->ok && (ov.path == 2 || ov.path == 4)) return EARS_ERR_SHAPE;   // the forced path cannot take this shape
    return EARS_OK;
}

int ensure_attrs(DeviceInfo* di) {
    static std::mutex attrs_mutex;   // two threads making their first call on a device set the attributes once
    std::lock_guard<std::mutex> lock(attrs_mutex);
    if (di->attrs_set) return EARS_OK;
    bool c16 = true;
    int rc = set_attrs<float>(&c16);
    if (rc) return rc;
    rc = set_attrs<uint16_t>(&c16);
    if (rc) return rc;
    rc = set_attrs<f16_t>(&c16);
    if (rc) return rc;
    di->cluster16 = c16;
    di->attrs_set = true;
    return EARS_OK;
}

// Everything about a call's arguments that the host can judge without a device.
int check_arguments(int dtype, const void* t, const void* d, const int32_t* x, int B, int K, int V,
                    float temperature, float beta, const float* seq_T, const float* seq_beta, unsigned flags,
                    int64_t b_first, const int32_t* out_len, const int32_t* out_tok) {
    if (!t || !d || !x || !out_len || !out_tok) return EARS_ERR_NULL;
    if (!dtype_ok(dtype)) return EARS_ERR_PARAM;
    if (flags & ~(unsigned)EARS_FLAGS_ALL) return EARS_ERR_PARAM;
    const int rc = check_shape(B, K, V);
    if (rc) return rc;
    // a per-sequence array replaces its scalar, which is then not looked at
    if (!seq_T && (!(temperature > 0.0f) || !std::isfinite(temperature))) return EARS_ERR_PARAM;
    if (!seq_beta && (!(beta >= 0.0f) || !std::isfinite(beta))) return EARS_ERR_PARAM;
    if (((uintptr_t)seq_T % 4) || ((uintptr_t)seq_beta % 4)) return EARS_ERR_ALIGN;
    if (b_first < 0 || (unsigned long long)b_first + (unsigned long long)B > 0xffffffffull) return EARS_ERR_PARAM;
    const int esize = dtype_size(dtype);
    if (((uintptr_t)t % esize) || ((uintptr_t)d % esize) || ((uintptr_t)x % 4)) return EARS_ERR_ALIGN;
    return EARS_OK;
}

int verify_impl(int dtype, const void* t, const void* d, const int32_t* x, int B, int K, int V,
                float temperature, float beta, const float* seq_T, const float* seq_beta, unsigned flags,
                uint64_t seed, uint64_t offset, int64_t b_first,
                int32_t* out_len, int32_t* out_tok, double* o_pt, double* o_pd, double* o_max,
                uint8_t* o_cls, double* o_resid, void* workspace, size_t workspace_bytes, void* stream_,
                double* o_entropy = nullptr) {
    int rc = check_arguments(dtype, t, d, x, B, K, V, temperature, beta, seq_T, seq_beta, flags, b_first, out_len, out_tok);
    if (rc) return rc;
    const int stop_first = (flags & EARS_FLAG_STOP_AT_FIRST_REJECT) ? 1 : 0;
    const int unc_entropy = (flags & EARS_FLAG_ENTROPY_UNCERTAINTY) ? 1 : 0;
    if (seq_T) temperature = 1.0f;
    if (seq_beta) beta = 0.0f;
    const int esize = dtype_size(dtype);
    if (workspace && ((uintptr_t)workspace % 256)) return EARS_ERR_ALIGN;
    if (!workspace && workspace_bytes != 0) return EARS_ERR_WORKSPACE;

    cudaStream_t stream = (cudaStream_t)stream_;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    DeviceInfo* di = nullptr;
    rc = device_info(dev, &di);
    if (rc) return rc;
    rc = ensure_attrs(di);
    if (rc) return rc;

    const bool aligned = ((uintptr_t)t % 16 == 0) && ((uintptr_t)d % 16 == 0) && (((size_t)V * esize) % 16 == 0);
    PlanOverride ov;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ov = g_override;
    }
    const float c = (float)(1.4426950408889634 / (double)temperature);

    // Rows small enough to stay in a cluster's shared memory take the resident path.
    RPlan rp;
    int max_clusters = 0;
    rc = choose_resident(dtype, B, K, V, stop_first != 0, di, ov, &rp, &max_clusters);
    if (rc) return rc;
    if (rp.ok) {
        const RLayout L = make_rlayout(B, K, V);
        if (workspace && workspace_bytes < L.total) return EARS_ERR_WORKSPACE;
        char *w = nullptr, *cw = nullptr;
        RParams p;
        rc = pick_counters(workspace, dev, stream_, 2, L.counters_bytes, L.total, &w, &cw, &p.zero_ptr, &p.zero_words);
        if (rc) return rc;
        p.t = t; p.d = d; p.x = x;
        p.B = B; p.K = K; p.V = V;
        p.c = c;
        p.T = (double)temperature;
        p.beta = (double)beta;
        p.seq_T = seq_T; p.seq_beta = seq_beta;
        p.seed = seed; p.offset = offset; p.b_first = b_first;
        p.out_len = out_len; p.out_tok = out_tok;
        p.pt_tok = o_pt ? o_pt : (double*)(w + L.pt_tok);
        p.pd_tok = o_pd ? o_pd : (double*)(w + L.pd_tok);
        p.max_pt = o_max ? o_max : (double*)(w + L.max_pt);
        p.cls = o_cls ? o_cls : (uint8_t*)(w + L.cls);
        p.resid = o_resid ? o_resid : (double*)(w + L.resid);
        p.heads = (int*)(cw + L.heads);
        p.ticket = (int*)(cw + L.ticket);
        p.flag = (signed char*)(w + L.flag);
        p.cand = (int32_t*)(w + L.cand);
        p.cand_mass = (double*)(w + L.cand_mass);
        p.rowstat = (float4*)(w + L.rowstat);
        p.seqmask = (unsigned long long*)(cw + L.seqmask);
        p.ready = (unsigned long long*)(cw + L.ready);
        p.ticket2 = (int*)(cw + L.ticket2);
        p.segsums = (double*)(w + L.seg);
        p.nseg = L.nseg;
        p.job_elems = rp.job_elems;
        p.parts2 = rp.parts2;
        p.C = rp.C; p.slice = rp.slice; p.buf_bytes = rp.buf_bytes;
        p.use_tma = aligned && ov.loader != 2;
        p.n_clusters = 0;
        p.want_stats = (o_pt || o_pd || o_max || o_cls) ? 1 : 0;
        p.ordered = stop_first;
        p.unc_entropy = unc_entropy;
        p.entropy = o_entropy;
        rc = by_dtype(dtype, [&](auto* e) {
            return launch_resident<std::remove_pointer_t<decltype(e)>>(p, rp, max_clusters, stream);
        });
        if (rc && !workspace) forget_clean_counters(dev, stream_);
        return rc;
    }

    // Long rows: 2-byte logits go to the kernel that reads straight from global memory (its warps
    // do not march in step, which the special-function pipe rewards), 4-byte logits to the kernel
    // with the shared-memory ring (HBM-bound either way; measured 570 against 592 us on B=512,
    // K=3, V=256000).  Path 1 / 3 force one or the other.
    const bool direct = use_direct(ov, esize, V, (long long)B * (K + 1));
    const Plan plan = make_plan(B, K, V, esize, aligned, di->sms, ov, direct);
    const Layout L = make_layout(B, K, V, plan.parts1);
    if (workspace && workspace_bytes < L.total) return EARS_ERR_WORKSPACE;
    char *w = nullptr, *cw = nullptr;
    Params p;
    rc = pick_counters(workspace, dev, stream_, 1, L.counters_bytes, L.total, &w, &cw, &p.zero_ptr, &p.zero_words);
    if (rc) return rc;

    p.t = t; p.d = d; p.x = x;
    p.B = B; p.K = K; p.V = V;
    p.c = c;
    p.T = (double)temperature;
    p.beta = (double)beta;
    p.seq_T = seq_T; p.seq_beta = seq_beta;
    p.seed = seed; p.offset = offset; p.b_first = b_first;
    p.out_len = out_len; p.out_tok = out_tok;
    p.pt_tok = o_pt ? o_pt : (double*)(w + L.pt_tok);
    p.pd_tok = o_pd ? o_pd : (double*)(w + L.pd_tok);
    p.max_pt = o_max ? o_max : (double*)(w + L.max_pt);
    p.cls = o_cls ? o_cls : (uint8_t*)(w + L.cls);
    p.resid = o_resid ? o_resid : (double*)(w + L.resid);
    p.ticket1 = (int*)(cw + L.ticket1);
    p.ticket_row = (int*)(cw + L.ticket_row);
    p.ticket2 = (int*)(cw + L.ticket2);
    p.job_ctr = (int*)(cw + L.job_ctr);
    p.ready = (unsigned long long*)(cw + L.ready);
    p.heads = (int*)(cw + L.heads);
    p.wq = (unsigned long long*)(cw + L.wq);
    p.partial = (float2*)(w + L.partial);
    p.rowstat = (float2*)(w + L.rowstat);
    p.seg_base = (unsigned char*)(w + L.seg);
    p.seg_stride = L.seg_stride;
    p.stop_first = stop_first;
    p.unc_entropy = unc_entropy;
    p.entropy = o_entropy;
    p.partial_w = (float*)(w + L.partial_w);
    p.roww = (float*)(w + L.roww);
    p.plan = plan;
    rc = by_dtype(dtype, [&](auto* e) { return launch<std::remove_pointer_t<decltype(e)>>(p, di->sms, direct, stream); });
    if (rc && !workspace) forget_clean_counters(dev, stream_);
    return rc;
}

size_t workspace_bound(int B, int K, int V) {
    PlanOverride ov;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ov = g_override;
    }
    size_t best = 0;
    // the piece count depends on the SM count and element size; take the largest over both
    // element sizes at a small and a large SM count (more SMs never ask for fewer pieces)
    const int sm_counts[2] = {1, 1024};
    for (int esize = 2; esize <= 4; esize += 2)
        for (int s = 0; s < 2; ++s) {
            const Plan pl = make_plan(B, K, V, esize, true, sm_counts[s], ov);
            const size_t tot = make_layout(B, K, V, pl.parts1).total;
            if (tot > best) best = tot;
        }
    const size_t res = make_rlayout(B, K, V).total;
    if (res > best) best = res;
    for (int esize = 2; esize <= 4; esize += 2)
        for (int s = 0; s < 2; ++s) {
            const size_t tot = make_glayout(B, K, V, esize, sm_counts[s]).total;
            if (tot > best) best = tot;
        }
    return best;
}

// Scratch of the allocation-free entry point.  Part of the library image: each GPU that
// loads the library carries it.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernels must be given the address that call returns.
static __device__ __align__(256) unsigned char g_noalloc_scratch[EARS_NOALLOC_SCRATCH_BYTES];
std::map<int, void*> g_noalloc_ptr;  // device -> device address of g_noalloc_scratch

int noalloc_scratch(int dev, void** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_noalloc_ptr.find(dev);
    if (it == g_noalloc_ptr.end()) {
        void* ptr = nullptr;
        EARS_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));  // for the current device
        if (!ptr || ((uintptr_t)ptr % 256)) return EARS_ERR_ALIGN;
        it = g_noalloc_ptr.emplace(dev, ptr).first;
    }
    *out = it->second;
    return EARS_OK;
}

// Self-test of the bounded wait: a barrier nobody ever arrives at.  The wait must give up after
// the limit, raise the abort flag and let the kernel return normally with the timeout bit set.
static __device__ int g_selftest_status;

__global__ void bounded_wait_kernel(unsigned long long limit_ns) {
    __shared__ alignas(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const bool ok = mbar_wait(&bar, 0, &abort_flag, limit_ns);   // every thread waits; all give up
    if (!ok && threadIdx.x == 0) atomicOr(&g_selftest_status, kDevTimeout);
}

__global__ void philox_kernel(const uint32_t* ctr_key, uint32_t* out, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t* c = ctr_key + (size_t)i * 6;
    U32x4 r = philox4x32_10(U32x4{c[0], c[1], c[2], c[3]}, c[4], c[5]);
    out[(size_t)i * 4 + 0] = r.w0;
    out[(size_t)i * 4 + 1] = r.w1;
    out[(size_t)i * 4 + 2] = r.w2;
    out[(size_t)i * 4 + 3] = r.w3;
}

int read_status(int* heads, cudaStream_t stream) {
    int status = 0;
    EARS_CUDA(cudaMemcpyAsync(&status, heads + 2, sizeof(int), cudaMemcpyDeviceToHost, stream));
    EARS_CUDA(cudaStreamSynchronize(stream));
    return status;
}


// ---- vocabulary-sharded verification (three local phases, see ears_shard.cuh) ----
constexpr long long kShardWarpRowBytes = 256 * 1024;   // rows up to this size may go one per warp

struct SLayout {
    int P, piece_elems, nseg;
    size_t counters_bytes, ticket_row, ticket_seq, partial, rowstat, sel, seg, total;
};

SLayout make_slayout(int B, int K, int Vs, int esize) {
    SLayout L;
    const long long rows = (long long)B * (2 * K + 1);
    // about a thousand units (a few per CTA of a full grid), pieces of at least 16 KB
    long long P = (1024 + rows - 1) / rows;
    const long long most = std::max<long long>(1, (long long)Vs * esize / 16384);
    P = std::max<long long>(1, std::min<long long>(std::min<long long>(P, most), 64));
    L.piece_elems = (int)((((long long)Vs + P - 1) / P + 255) / 256 * 256);
    L.P = (Vs + L.piece_elems - 1) / L.piece_elems;
    L.nseg = (Vs + kSegElems - 1) / kSegElems;
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    size_t o = 0;
    L.ticket_row = o; o = up(o + (size_t)rows * 4);
    L.ticket_seq = o; o = up(o + (size_t)B * 4);
    L.counters_bytes = o;
    L.partial = o; o = up(o + (size_t)rows * L.P * 8);
    L.rowstat = o; o = up(o + (size_t)rows * 16);
    L.sel = o; o = up(o + (size_t)B * 4);
    L.seg = o; o = up(o + (size_t)B * L.nseg * 8);
    L.total = o;
    return L;
}

int shard_common(int dtype, const void* t, const void* d, const int32_t* x, int B, int K, int Vs, int V, int v_first,
                 int n_shards, int shard, float temperature, void* workspace, size_t workspace_bytes, SParams* p, SLayout* L,
                 DeviceInfo** di) {
    if (!t || !d || !x || !workspace) return EARS_ERR_NULL;
    if (!dtype_ok(dtype)) return EARS_ERR_PARAM;
    int rc = check_shape(B, K, Vs);
    if (rc) return rc;
    if (V < Vs || V > (1 << 30) || v_first < 0 || v_first > V - Vs) return EARS_ERR_SHAPE;
    if (n_shards < 1 || n_shards > EARS_MAX_SHARDS || shard < 0 || shard >= n_shards) return EARS_ERR_PARAM;
    if (!(temperature > 0.0f) || !std::isfinite(temperature)) return EARS_ERR_PARAM;
    const int esize = dtype_size(dtype);
    if (((uintptr_t)t % esize) || ((uintptr_t)d % esize) || ((uintptr_t)x % 4) || ((uintptr_t)workspace % 256)) return EARS_ERR_ALIGN;
    *L = make_slayout(B, K, Vs, esize);
    if (workspace_bytes < L->total) return EARS_ERR_WORKSPACE;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    rc = device_info(dev, di);
    if (rc) return rc;
    char* w = (char*)workspace;
    *p = SParams();
    p->t = t; p->d = d; p->x = x;
    p->B = B; p->K = K; p->Vs = Vs; p->V = V; p->v_first = v_first; p->n_shards = n_shards;
    p->P = L->P; p->piece_elems = L->piece_elems;
    p->vec = ((uintptr_t)t % 16 == 0) && ((uintptr_t)d % 16 == 0) && (((size_t)Vs * esize) % 16 == 0);
    p->c = (float)(1.4426950408889634 / (double)temperature);
    p->T = (double)temperature;
    p->ticket_row = (int*)(w + L->ticket_row);
    p->ticket_seq = (int*)(w + L->ticket_seq);
    p->partial = (float2*)(w + L->partial);
    p->rowstat = (float4*)(w + L->rowstat);
    p->sel = (int*)(w + L->sel);
    p->seg = (double*)(w + L->seg);
    p->nseg = L->nseg;
    return EARS_OK;
}

}  // namespace

extern "C" {

int ears_verify_ex(int dtype, const void* target_logits, const void* draft_logits,
                   const int32_t* draft_tokens, int B, int K, int V, float temperature, float beta,
                   uint64_t seed, uint64_t offset, int64_t b_first, int32_t* out_accept_len,
                   int32_t* out_tokens, double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                   uint8_t* out_class, double* out_resid_mass, void* workspace, size_t workspace_bytes,
                   void* stream) {
    return verify_impl(dtype, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta, nullptr, nullptr, 0u,
                       seed, offset, b_first, out_accept_len, out_tokens, out_pt_tok, out_pd_tok, out_max_pt,
                       out_class, out_resid_mass, workspace, workspace_bytes, stream);
}

int ears_verify_var(int dtype, const void* target_logits, const void* draft_logits,
                    const int32_t* draft_tokens, int B, int K, int V, float temperature, float beta,
                    const float* seq_temperature, const float* seq_beta, unsigned flags,
                    uint64_t seed, uint64_t offset, int64_t b_first, int32_t* out_accept_len,
                    int32_t* out_tokens, double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                    uint8_t* out_class, double* out_resid_mass, void* workspace, size_t workspace_bytes,
                    void* stream) {
    return verify_impl(dtype, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta,
                       seq_temperature, seq_beta, flags, seed, offset, b_first, out_accept_len, out_tokens, out_pt_tok,
                       out_pd_tok, out_max_pt, out_class, out_resid_mass, workspace, workspace_bytes, stream);
}

int ears_verify_entropy(int dtype, const void* target_logits, const void* draft_logits,
                        const int32_t* draft_tokens, int B, int K, int V, float temperature, float beta,
                        const float* seq_temperature, const float* seq_beta, unsigned flags,
                        uint64_t seed, uint64_t offset, int64_t b_first, int32_t* out_accept_len,
                        int32_t* out_tokens, double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                        uint8_t* out_class, double* out_resid_mass, double* out_entropy,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if ((uintptr_t)out_entropy % 8) return EARS_ERR_ALIGN;
    return verify_impl(dtype, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta,
                       seq_temperature, seq_beta, flags, seed, offset, b_first, out_accept_len, out_tokens, out_pt_tok,
                       out_pd_tok, out_max_pt, out_class, out_resid_mass, workspace, workspace_bytes, stream, out_entropy);
}

int ears_verify_greedy(int dtype, const void* target_logits, const int32_t* draft_tokens, int B, int K, int V,
                       int32_t* out_accept_len, int32_t* out_tokens, void* workspace, size_t workspace_bytes,
                       void* stream_) {
    if (!target_logits || !draft_tokens || !out_accept_len || !out_tokens) return EARS_ERR_NULL;
    if (!dtype_ok(dtype)) return EARS_ERR_PARAM;
    int rc = check_shape(B, K, V);
    if (rc) return rc;
    const int esize = dtype_size(dtype);
    if (((uintptr_t)target_logits % esize) || ((uintptr_t)draft_tokens % 4)) return EARS_ERR_ALIGN;
    if (workspace && ((uintptr_t)workspace % 256)) return EARS_ERR_ALIGN;
    if (!workspace && workspace_bytes != 0) return EARS_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    DeviceInfo* di = nullptr;
    rc = device_info(dev, &di);
    if (rc) return rc;
    const GLayout L = make_glayout(B, K, V, esize, di->sms);
    if (workspace && workspace_bytes < L.total) return EARS_ERR_WORKSPACE;
    GParams p;
    char *w = nullptr, *cw = nullptr;
    rc = pick_counters(workspace, dev, stream_, 3, L.counters_bytes, L.total, &w, &cw, &p.zero_ptr, &p.zero_words);
    if (rc) return rc;
    p.t = target_logits; p.x = draft_tokens;
    p.B = B; p.K = K; p.V = V;
    p.P = L.P; p.piece_elems = L.piece_elems;
    p.vec = ((uintptr_t)target_logits % 16 == 0) && (((size_t)V * esize) % 16 == 0);
    p.units = (long long)B * (K + 1) * L.P;
    p.partial = (int4*)(w + L.partial);
    p.ticket = (int*)(cw + L.ticket);
    p.heads = (int*)(cw + L.heads);
    p.out_len = out_accept_len; p.out_tok = out_tokens;
    const long long cap = (long long)kGCtasPerSm * di->sms;
    const int grid = (int)(p.units < cap ? p.units : cap);
    const bool timed = profile_wanted();
    rc = profile_mark(stream, timed);
    if (rc) return rc;
    by_dtype(dtype, [&](auto* e) {
        ears_greedy_kernel<std::remove_pointer_t<decltype(e)>><<<grid, kGThreads, 0, stream>>>(p);
        return 0;
    });
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        if (!workspace) forget_clean_counters(dev, stream_);
        return cuda_fail(e, "ears_greedy_kernel launch");
    }
    return profile_mark(stream, timed);
}

int ears_verify_f32(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                    int B, int K, int V, float temperature, float beta, uint64_t seed, uint64_t offset,
                    int32_t* out_accept_len, int32_t* out_tokens, void* stream) {
    return verify_impl(EARS_DTYPE_F32, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta,
                       nullptr, nullptr, 0u, seed, offset, 0, out_accept_len, out_tokens, nullptr, nullptr, nullptr, nullptr, nullptr,
                       nullptr, 0, stream);
}

int ears_verify_bf16(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                     int B, int K, int V, float temperature, float beta, uint64_t seed, uint64_t offset,
                     int32_t* out_accept_len, int32_t* out_tokens, void* stream) {
    return verify_impl(EARS_DTYPE_BF16, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta,
                       nullptr, nullptr, 0u, seed, offset, 0, out_accept_len, out_tokens, nullptr, nullptr, nullptr, nullptr, nullptr,
                       nullptr, 0, stream);
}

int ears_verify_f16(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                    int B, int K, int V, float temperature, float beta, uint64_t seed, uint64_t offset,
                    int32_t* out_accept_len, int32_t* out_tokens, void* stream) {
    return verify_impl(EARS_DTYPE_F16, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta,
                       nullptr, nullptr, 0u, seed, offset, 0, out_accept_len, out_tokens, nullptr, nullptr, nullptr, nullptr, nullptr,
                       nullptr, 0, stream);
}

int ears_verify(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                int B, int K, int V, float temperature, float beta, uint64_t seed, uint64_t offset,
                int32_t* out_accept_len, int32_t* out_tokens, void* stream) {
    return ears_verify_f32((const float*)target_logits, (const float*)draft_logits, draft_tokens, B, K, V,
                           temperature, beta, seed, offset, out_accept_len, out_tokens, stream);
}

int ears_verify_host(int dtype, const void* target_logits, const void* draft_logits,
                     const int32_t* draft_tokens, int B, int K, int V, float temperature, float beta,
                     uint64_t seed, uint64_t offset, int64_t b_first, int32_t* out_accept_len,
                     int32_t* out_tokens, void* stream_) {
    if (!target_logits || !draft_logits || !draft_tokens || !out_accept_len || !out_tokens) return EARS_ERR_NULL;
    if (!dtype_ok(dtype)) return EARS_ERR_PARAM;
    int rc = check_shape(B, K, V);
    if (rc) return rc;
    const size_t esize = (size_t)dtype_size(dtype);
    const size_t tb = (size_t)B * (K + 1) * V * esize, db = (size_t)B * K * V * esize;
    const size_t xb = (size_t)B * K * 4, lb = (size_t)B * 4, ob = (size_t)B * (K + 1) * 4;
    size_t o_t = 0, o_d = align_up(o_t + tb, 256), o_x = align_up(o_d + db, 256);
    size_t o_l = align_up(o_x + xb, 256), o_o = align_up(o_l + lb, 256), total = align_up(o_o + ob, 256);
    cudaStream_t stream = (cudaStream_t)stream_;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    void* base = nullptr;
    rc = get_buffer(g_staging, dev, stream_, total, &base);
    if (rc) return rc;
    char* s = (char*)base;
    EARS_CUDA(cudaMemcpyAsync(s + o_t, target_logits, tb, cudaMemcpyHostToDevice, stream));
    EARS_CUDA(cudaMemcpyAsync(s + o_d, draft_logits, db, cudaMemcpyHostToDevice, stream));
    EARS_CUDA(cudaMemcpyAsync(s + o_x, draft_tokens, xb, cudaMemcpyHostToDevice, stream));
    rc = verify_impl(dtype, s + o_t, s + o_d, (const int32_t*)(s + o_x), B, K, V, temperature, beta, nullptr, nullptr, 0u,
                     seed, offset, b_first, (int32_t*)(s + o_l), (int32_t*)(s + o_o), nullptr, nullptr, nullptr, nullptr,
                     nullptr, nullptr, 0, stream_);
    if (rc) return rc;
    EARS_CUDA(cudaMemcpyAsync(out_accept_len, s + o_l, lb, cudaMemcpyDeviceToHost, stream));
    EARS_CUDA(cudaMemcpyAsync(out_tokens, s + o_o, ob, cudaMemcpyDeviceToHost, stream));
    const int status = ears_last_device_status(stream_);
    if (status < 0) return status;
    return (status & EARS_DEV_TIMEOUT) ? EARS_ERR_TIMEOUT : EARS_OK;
}

int ears_verify_noalloc(int dtype, const void* target_logits, const void* draft_logits,
                        const int32_t* draft_tokens, int B, int K, int V, float temperature, float beta,
                        uint64_t seed, uint64_t offset, int64_t b_first, int32_t* out_accept_len,
                        int32_t* out_tokens, int32_t* out_device_status, void* stream) {
    // what the host can judge comes first: a bad argument is reported as such, device or no device
    int rc = check_arguments(dtype, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta, nullptr, nullptr,
                             0u, b_first, out_accept_len, out_tokens);
    if (rc) return rc;
    if (workspace_bound(B, K, V) > (size_t)EARS_NOALLOC_SCRATCH_BYTES) return EARS_ERR_WORKSPACE;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    void* scratch = nullptr;
    rc = noalloc_scratch(dev, &scratch);
    if (rc) return rc;
    rc = verify_impl(dtype, target_logits, draft_logits, draft_tokens, B, K, V, temperature, beta, nullptr, nullptr, 0u,
                     seed, offset, b_first, out_accept_len, out_tokens, nullptr, nullptr, nullptr, nullptr, nullptr, scratch,
                     (size_t)EARS_NOALLOC_SCRATCH_BYTES, stream);
    if (rc) return rc;
    if (out_device_status)  // the status word is heads[2] at the start of the scratch
        EARS_CUDA(cudaMemcpyAsync(out_device_status, (const int*)scratch + 2, sizeof(int),
                                  cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return EARS_OK;
}

size_t ears_workspace_bytes(int B, int K, int V) {
    if (check_shape(B, K, V)) return 0;
    return workspace_bound(B, K, V);
}

int ears_last_device_status(void* stream_) {
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    void* word = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        auto it = g_workspaces.find(std::make_pair(dev, stream_));
        if (it != g_workspaces.end()) word = it->second.status_word;
    }
    if (!word) {
        EARS_CUDA(cudaStreamSynchronize((cudaStream_t)stream_));
        return 0;
    }
    return read_status((int*)word - 2, (cudaStream_t)stream_);
}

int ears_workspace_device_status(void* workspace, void* stream_) {
    if (!workspace) return EARS_ERR_NULL;
    return read_status((int*)workspace, (cudaStream_t)stream_);
}

static int read_counts(const int* heads, cudaStream_t stream, uint32_t out_counts[4]) {
    EARS_CUDA(cudaMemcpyAsync(out_counts, heads + kCountDirect, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    EARS_CUDA(cudaStreamSynchronize(stream));
    return EARS_OK;
}

int ears_last_decision_counts(void* stream_, uint32_t out_counts[4]) {
    if (!out_counts) return EARS_ERR_NULL;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    void* word = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        auto it = g_workspaces.find(std::make_pair(dev, stream_));
        if (it != g_workspaces.end()) word = it->second.status_word;
    }
    out_counts[0] = out_counts[1] = out_counts[2] = out_counts[3] = 0;
    if (!word) {
        EARS_CUDA(cudaStreamSynchronize((cudaStream_t)stream_));
        return EARS_OK;
    }
    return read_counts((const int*)word - 2, (cudaStream_t)stream_, out_counts);
}

int ears_workspace_decision_counts(void* workspace, void* stream_, uint32_t out_counts[4]) {
    if (!workspace || !out_counts) return EARS_ERR_NULL;
    return read_counts((const int*)workspace, (cudaStream_t)stream_, out_counts);
}

int ears_selftest_bounded_wait(int limit_ms, void* stream_) {
    if (limit_ms < 1 || limit_ms > 2000) return EARS_ERR_PARAM;
    cudaStream_t stream = (cudaStream_t)stream_;
    int seen = 0;
    EARS_CUDA(cudaMemcpyToSymbolAsync(g_selftest_status, &seen, sizeof(int), 0, cudaMemcpyHostToDevice, stream));
    bounded_wait_kernel<<<1, 64, 0, stream>>>((unsigned long long)limit_ms * 1000000ull);
    EARS_CUDA(cudaGetLastError());
    EARS_CUDA(cudaMemcpyFromSymbolAsync(&seen, g_selftest_status, sizeof(int), 0, cudaMemcpyDeviceToHost, stream));
    EARS_CUDA(cudaStreamSynchronize(stream));
    return (seen & EARS_DEV_TIMEOUT) ? EARS_ERR_TIMEOUT : EARS_OK;
}

int ears_philox_device(const uint32_t* ctr_key, uint32_t* out, int n, void* stream) {
    if (n < 0) return EARS_ERR_SHAPE;
    if (n == 0) return EARS_OK;
    if (!ctr_key || !out) return EARS_ERR_NULL;
    philox_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(ctr_key, out, n);
    EARS_CUDA(cudaGetLastError());
    return EARS_OK;
}

int ears_set_plan(int loader, int parts) {
    if (loader < 0 || loader > 2 || parts < 0) return EARS_ERR_PARAM;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_override.loader = loader;
    g_override.parts1 = parts;
    return EARS_OK;
}

int ears_describe_plan(int dtype, int B, int K, int V, char* out, size_t out_bytes) {
    if (!out || out_bytes == 0) return EARS_ERR_NULL;
    if (!dtype_ok(dtype)) return EARS_ERR_PARAM;
    int rc = check_shape(B, K, V);
    if (rc) return rc;
    int dev = 0;
    EARS_CUDA(cudaGetDevice(&dev));
    DeviceInfo* di = nullptr;
    rc = device_info(dev, &di);
    if (rc) return rc;
    rc = ensure_attrs(di);
    if (rc) return rc;
    PlanOverride ov;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ov = g_override;
    }
    RPlan rp;
    int max_clusters = 0;
    rc = choose_resident(dtype, B, K, V, false, di, ov, &rp, &max_clusters);
    if (rc) return rc;
    const int esize = dtype_size(dtype);
    if (rp.ok) {
        const long long items = (long long)B * (K + 1);
        int per_sm = 0;
        by_dtype(dtype, [&](auto* e) {
            using El = std::remove_pointer_t<decltype(e)>;
            return rp.streamed ? (int)cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ears_cstream_kernel<El, false>, kCThreads, rp.smem)
                               : (int)cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ears_resident_kernel<El, false>, kRThreads, rp.smem);
        });
        if (rp.streamed)
            snprintf(out, out_bytes, "cluster-streamed: cluster=%d slice_elems=%d smem_bytes=%zu ctas_per_sm=%d clusters_resident=%d clusters_launched=%lld second_pass_pieces=%d",
                     rp.C, rp.slice, rp.smem, per_sm, max_clusters, items < max_clusters ? items : (long long)max_clusters, rp.parts2);
        else
            snprintf(out, out_bytes, "resident: cluster=%d slice_elems=%d smem_bytes=%zu ctas_per_sm=%d clusters_resident=%d clusters_launched=%lld",
                     rp.C, rp.slice, rp.smem, per_sm, max_clusters, items < max_clusters ? items : (long long)max_clusters);
    } else {
        const bool direct = use_direct(ov, esize, V, (long long)B * (K + 1));
        const Plan pl = make_plan(B, K, V, esize, true, di->sms, ov, direct);
        const long long units = (long long)B * (2 * K + 1) * pl.parts1, cap = (long long)di->sms * kCtasPerSm;
        if (!direct) {
            snprintf(out, out_bytes, "streaming: pieces_per_row=%d chunks_per_piece=%d ctas=%lld second_pass_pieces=%d",
                     pl.parts1, pl.cpp1, units < cap ? units : cap, pl.parts2);
        } else {
            const long long dcap = (long long)di->sms * kDCtasPerSm;
            snprintf(out, out_bytes, "direct: pieces_per_row=%d chunks_per_piece=%d ctas=%lld second_pass_pieces=%d",
                     pl.parts1, pl.cpp1, units < dcap ? units : dcap, pl.parts2);
        }
    }
    return EARS_OK;
}

int ears_set_path(int path, int cluster) {
    if (path < 0 || path > 4) return EARS_ERR_PARAM;
    if (cluster != 0 && cluster != 1 && cluster != 2 && cluster != 4 && cluster != 8 && cluster != 16) return EARS_ERR_PARAM;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_override.path = path;
    g_override.cluster = cluster;
    return EARS_OK;
}

int ears_profile_begin(int max_calls) {
    if (max_calls < 1 || max_calls > (1 << 16)) return EARS_ERR_PARAM;
    for (cudaEvent_t ev : g_profile.events) cudaEventDestroy(ev);
    g_profile.events.clear();
    g_profile.used = 0;
    g_profile.active = false;
    // all events are created here, so that a timed call adds two cudaEventRecord and nothing else
    g_profile.events.reserve((size_t)2 * max_calls);
    for (int i = 0; i < 2 * max_calls; ++i) {
        cudaEvent_t ev;
        EARS_CUDA(cudaEventCreate(&ev));
        g_profile.events.push_back(ev);
    }
    g_profile.max_calls = max_calls;
    g_profile.active = true;
    return EARS_OK;
}

int ears_profile_end(float* kernel_ms, int capacity, int* n_calls) {
    if (!kernel_ms || !n_calls) return EARS_ERR_NULL;
    g_profile.active = false;
    const int calls = (int)(g_profile.used / 2);
    int rc = EARS_OK;
    if (calls > 0) {
        cudaError_t e = cudaEventSynchronize(g_profile.events[(size_t)2 * calls - 1]);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaEventSynchronize");
    }
    int n = 0;
    for (int i = 0; i < calls && i < capacity && rc == EARS_OK; ++i, ++n) {
        cudaError_t e = cudaEventElapsedTime(&kernel_ms[i], g_profile.events[2 * i], g_profile.events[2 * i + 1]);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaEventElapsedTime");
    }
    for (cudaEvent_t ev : g_profile.events) cudaEventDestroy(ev);
    g_profile.events.clear();
    g_profile.used = 0;
    *n_calls = n;
    return rc;
}

const char* ears_status_string(int status) {
    switch (status) {
        case EARS_OK: return "ok";
        case EARS_ERR_NULL: return "a required pointer is NULL";
        case EARS_ERR_SHAPE: return "B, K or V out of range";
        case EARS_ERR_PARAM: return "bad temperature, beta, dtype or sequence offset";
        case EARS_ERR_ALIGN: return "pointer not aligned";
        case EARS_ERR_WORKSPACE: return "workspace too small";
        case EARS_ERR_CUDA: return "a CUDA call failed";
        case EARS_ERR_TIMEOUT: return "a device-side wait timed out";
        default: return "unknown status";
    }
}

size_t ears_shard_workspace_bytes(int dtype, int B, int K, int Vs) {
    if (!dtype_ok(dtype) || check_shape(B, K, Vs)) return 0;
    return make_slayout(B, K, Vs, dtype_size(dtype)).total;
}

int ears_shard_stats(int dtype, const void* target_shard, const void* draft_shard, const int32_t* draft_tokens,
                     int B, int K, int Vs, int V, int v_first, float temperature, float* out_stats,
                     void* workspace, size_t workspace_bytes, void* stream_) {
    if (!out_stats) return EARS_ERR_NULL;
    if ((uintptr_t)out_stats % 16) return EARS_ERR_ALIGN;
    SParams p; SLayout L; DeviceInfo* di = nullptr;
    int rc = shard_common(dtype, target_shard, draft_shard, draft_tokens, B, K, Vs, V, v_first, 1, 0, temperature,
                          workspace, workspace_bytes, &p, &L, &di);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    p.stats = (float4*)out_stats;
    const long long rows = (long long)B * (2 * K + 1), cap = (long long)kSCtasPerSm * di->sms;
    if (L.P == 1 && (long long)Vs * dtype_size(dtype) <= kShardWarpRowBytes && rows >= 2 * cap * (kSThreads / 32)) {
        // many short rows (several rounds of one row per warp): a warp per row
        const long long want = (rows + kSThreads / 32 - 1) / (kSThreads / 32);
        const int grid = (int)(want < cap ? want : cap);
        by_dtype(dtype, [&](auto* e) {
            ears_shard_stats_rows_kernel<std::remove_pointer_t<decltype(e)>><<<grid, kSThreads, 0, stream>>>(p);
            return 0;
        });
    } else {
        EARS_CUDA(cudaMemsetAsync(p.ticket_row, 0, (size_t)rows * 4, stream));
        const long long units = rows * L.P;
        const int grid = (int)(units < cap ? units : cap);
        by_dtype(dtype, [&](auto* e) {
            ears_shard_stats_kernel<std::remove_pointer_t<decltype(e)>><<<grid, kSThreads, 0, stream>>>(p);
            return 0;
        });
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ears_shard_stats_kernel launch");
    return EARS_OK;
}

int ears_shard_decide(int dtype, const void* target_shard, const void* draft_shard, const int32_t* draft_tokens,
                      int B, int K, int Vs, int V, int v_first, int n_shards, const float* all_stats,
                      float temperature, float beta, uint64_t seed, uint64_t offset, int64_t b_first,
                      int32_t* out_accept_len, int32_t* out_tokens, double* out_mass,
                      void* workspace, size_t workspace_bytes, void* stream_) {
    if (!all_stats || !out_accept_len || !out_tokens || !out_mass) return EARS_ERR_NULL;
    if (((uintptr_t)all_stats % 16) || ((uintptr_t)out_mass % 8)) return EARS_ERR_ALIGN;
    if (!(beta >= 0.0f) || !std::isfinite(beta)) return EARS_ERR_PARAM;
    if (b_first < 0 || (unsigned long long)b_first + (unsigned long long)B > 0xffffffffull) return EARS_ERR_PARAM;
    SParams p; SLayout L; DeviceInfo* di = nullptr;
    int rc = shard_common(dtype, target_shard, draft_shard, draft_tokens, B, K, Vs, V, v_first, n_shards, 0, temperature,
                          workspace, workspace_bytes, &p, &L, &di);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    p.all_stats = (const float4*)all_stats;
    p.beta = (double)beta;
    p.seed = seed; p.offset = offset; p.b_first = b_first;
    p.out_len = out_accept_len; p.out_tok = out_tokens; p.mass = out_mass;
    EARS_CUDA(cudaMemsetAsync(p.ticket_seq, 0, (size_t)B * 4, stream));
    ears_shard_decide_kernel<<<(B + kSSeqPerCta - 1) / kSSeqPerCta, kSSeqPerCta * 32, 0, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ears_shard_decide_kernel launch");
    const int cps = (L.nseg + kSSegsPerCta - 1) / kSSegsPerCta;
    if ((long long)B * cps > 0x7fffffffll) return EARS_ERR_SHAPE;
    by_dtype(dtype, [&](auto* el) {
        ears_shard_mass_kernel<std::remove_pointer_t<decltype(el)>><<<B * cps, kSThreads, 0, stream>>>(p, cps);
        return 0;
    });
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ears_shard_mass_kernel launch");
    return EARS_OK;
}

int ears_shard_pick(int dtype, const void* target_shard, const void* draft_shard, const int32_t* draft_tokens,
                    int B, int K, int Vs, int V, int v_first, int n_shards, int shard, const float* all_stats,
                    const double* all_mass, float temperature, uint64_t seed, uint64_t offset, int64_t b_first,
                    int32_t* out_tokens, void* workspace, size_t workspace_bytes, void* stream_) {
    if (!all_stats || !all_mass || !out_tokens) return EARS_ERR_NULL;
    if (((uintptr_t)all_stats % 16) || ((uintptr_t)all_mass % 8)) return EARS_ERR_ALIGN;
    if (b_first < 0 || (unsigned long long)b_first + (unsigned long long)B > 0xffffffffull) return EARS_ERR_PARAM;
    SParams p; SLayout L; DeviceInfo* di = nullptr;
    int rc = shard_common(dtype, target_shard, draft_shard, draft_tokens, B, K, Vs, V, v_first, n_shards, shard, temperature,
                          workspace, workspace_bytes, &p, &L, &di);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    p.all_stats = (const float4*)all_stats;
    p.all_mass = all_mass;
    p.seed = seed; p.offset = offset; p.b_first = b_first;
    p.out_tok = out_tokens;
    by_dtype(dtype, [&](auto* el) {
        ears_shard_pick_kernel<std::remove_pointer_t<decltype(el)>>
            <<<(B + kSSeqPerCta - 1) / kSSeqPerCta, kSSeqPerCta * 32, 0, stream>>>(p, shard);
        return 0;
    });
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ears_shard_pick_kernel launch");
    return EARS_OK;
}

#ifdef EARS_TRACE
// Timeline build only (not part of the public header): clears, then reads back, what the kernels' marks recorded.
int ears_trace_reset(void) {
    static int zeros[kTraceCtas];
    EARS_CUDA(cudaMemcpyToSymbol(g_trace_n, zeros, sizeof zeros));
    return EARS_OK;
}
// out: [kTraceCtas][kTraceEvents][2] 64-bit words (time in ns; tag << 32 | argument); counts: [kTraceCtas]
int ears_trace_read(unsigned long long* out, int* counts, int* n_ctas, int* n_events) {
    EARS_CUDA(cudaDeviceSynchronize());
    EARS_CUDA(cudaMemcpyFromSymbol(out, g_trace, sizeof(unsigned long long) * kTraceCtas * kTraceEvents * 2));
    EARS_CUDA(cudaMemcpyFromSymbol(counts, g_trace_n, sizeof(int) * kTraceCtas));
    *n_ctas = kTraceCtas;
    *n_events = kTraceEvents;
    return EARS_OK;
}
#endif

const char* ears_last_cuda_error(void) { return g_cuda_error; }

int ears_version(void) { return EARS_VERSION; }

void ears_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int cur = 0;
    cudaGetDevice(&cur);
    for (auto* pool : {&g_workspaces, &g_staging}) {
        for (auto& kv : *pool) {
            if (!kv.second.ptr) continue;
            cudaSetDevice(kv.first.first);
            cudaDeviceSynchronize();
            cudaFree(kv.second.ptr);
        }
        pool->clear();
    }
    for (auto& dp : g_parked) {
        cudaSetDevice(dp.first);
        cudaDeviceSynchronize();
        cudaFree(dp.second);
    }
    g_parked.clear();
    cudaSetDevice(cur);
}

}  // extern "C"
