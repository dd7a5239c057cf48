// Shared-memory pipeline primitives for sm_100a: mbarrier wrappers with bounded
// waits and the 1-D bulk asynchronous copy (TMA, each CTA for itself) that feeds the
// streaming kernels.  Every wait gives up after a time limit, records it in a
// block-wide abort flag and lets the caller unwind; nothing here can spin forever.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace ears {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait before giving up
// How long one try_wait may keep the warp suspended in hardware before it reports "not yet":
// long enough that a waiting warp issues almost nothing, short against the limit above.
constexpr unsigned kTryWaitHintNs = 20000;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// ---- optional timeline (compiled in with -DEARS_TRACE only) ----------------------------
// A few CTAs record (time, tag, argument) at the ends of their phases into a fixed device array
// that the host reads back with ears_trace_read; used to see where a launch spends its time.
// Without the macro the marks compile to nothing.
#ifdef EARS_TRACE
constexpr int kTraceCtas = 96, kTraceEvents = 192;
__device__ unsigned long long g_trace[kTraceCtas][kTraceEvents][2];
__device__ int g_trace_n[kTraceCtas];
// called by one thread of the CTA
__device__ __forceinline__ void trace_mark(int tag, int arg) {
    if (blockIdx.x < kTraceCtas) {
        const int i = g_trace_n[blockIdx.x]++;
        if (i < kTraceEvents) {
            g_trace[blockIdx.x][i][0] = global_timer_ns();
            g_trace[blockIdx.x][i][1] = ((unsigned long long)(unsigned)tag << 32) | (unsigned)arg;
        }
    }
}
#else
__device__ __forceinline__ void trace_mark(int, int) {}
#endif

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous (TMA) proxy.
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kTryWaitHintNs)
        : "memory");
    return ok != 0;
}

// Waits for the phase with the given parity.  Returns false if the block is
// aborting or the time limit passed (then it also raises the abort flag).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs) {
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
        }
    }
}

// global -> this CTA's shared memory, completion counted in bytes on `bar`.
// dst, src and bytes must be multiples of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// Same copy with an L2 eviction-priority hint (a policy made by l2_policy_*).
__device__ __forceinline__ void bulk_load_hint(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// Counts an arrival with release + acquire semantics at device scope in the atomic itself:
// what this thread wrote (or observed) before is visible to whoever sees the count, and what
// earlier arrivals published is visible to this thread afterwards.  One round trip, no fence.
__device__ __forceinline__ int ticket_add(int* addr) {
    int old;
    asm volatile("atom.add.acq_rel.gpu.s32 %0, [%1], 1;" : "=r"(old) : "l"(addr) : "memory");
    return old;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

// IEEE binary16 logits: a 2-byte element type of its own (uint16_t stands for bfloat16 bits).
struct f16_t { uint16_t bits; };

// both halves of a packed pair -> fp32 (exact)
__device__ __forceinline__ float2 f16x2_to_float2(uint32_t w) {
    float lo, hi;
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}"
        : "=f"(lo), "=f"(hi) : "r"(w));
    return make_float2(lo, hi);
}
// one element through the read-only path, unconverted
__device__ __forceinline__ float ld_elem(const float* p) { return __ldg(p); }
__device__ __forceinline__ uint16_t ld_elem(const uint16_t* p) { return __ldg(p); }
__device__ __forceinline__ f16_t ld_elem(const f16_t* p) { f16_t r; r.bits = __ldg(&p->bits); return r; }

__device__ __forceinline__ float f16_bits_to_float(uint16_t bits) {
    float r;
    asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(bits));
    return r;
}

// (m, s) pairs describe sum_v exp2((l_v - m) * c) = s.  Merging keeps the larger m.
// -inf maxima (nothing finite seen yet) contribute nothing; NaN sums propagate.
__device__ __forceinline__ void merge_ms(float& m, float& s, float m2, float s2, float c) {
    float mn = fmaxf(m, m2);
    if (mn == -INFINITY) { s = s + s2; return; }  // both empty (sums are 0 unless NaN)
    // full-precision exp2 (one of the two factors is exactly 1): merges happen once per piece, and
    // the error of an approximate factor would be common to everything merged so far
    float a = exp2f((m - mn) * c);                // (-inf - finite) -> 0
    float b = exp2f((m2 - mn) * c);
    s = s * a + s2 * b;
    m = mn;
}

}  // namespace ears
