// Arithmetic shared by the verification kernels: unpacking of staged logits, the mass of one
// vocabulary entry in the final draw, and the per-position decision of Sec. 3.2.
#pragma once
#include "ears_common.cuh"
#include "ears_pipeline.cuh"

namespace ears {

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
template <> struct Vec<f16_t> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void unpack(uint4 v, float (&x)[8]) {
        const float2 a = f16x2_to_float2(v.x), b = f16x2_to_float2(v.y), c = f16x2_to_float2(v.z), d = f16x2_to_float2(v.w);
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y; x[4] = c.x; x[5] = c.y; x[6] = d.x; x[7] = d.y;
    }
    __device__ static __forceinline__ void load(const unsigned char* buf, int vec_index, float (&x)[8]) {
        unpack(reinterpret_cast<const uint4*>(buf)[vec_index], x);
    }
};

__device__ __forceinline__ float load_logit(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_logit(const uint16_t* p) { return bf16_bits_to_float(__ldg(p)); }
__device__ __forceinline__ float load_logit(const f16_t* p) { return f16_bits_to_float(__ldg(&p->bits)); }

struct RowNorm {
    float mt, md;          // row maxima
    float rho_hi, rho_lo;  // Z_t / Z_d split in two floats (residual rows)
    double izt;            // 1 / Z_t
};

__device__ __forceinline__ RowNorm make_rownorm(float2 st, float2 sd) {
    const double rho = (double)st.y / (double)sd.y;
    const float hi = (float)rho;
    return RowNorm{st.x, sd.x, hi, (float)(rho - (double)hi), 1.0 / (double)st.y};
}

// Mass of one vocabulary entry for the final draw in units of 1/Z_t:
// Z_t P_t(v), or Z_t max(0, P_t(v) - P_d(v)) = max(0, e_t - e_d Z_t/Z_d).  The common factor
// cancels in the inverse-CDF draw.  fp32 with the ratio carried as hi + lo so that no
// systematic rounding of Z_t/Z_d tilts the residual; explicit rounding intrinsics so that the
// streaming pass and the in-segment pass produce identical bits.
template <bool RESID>
__device__ __forceinline__ float entry_mass(float xt, float xd, const RowNorm& rn, float c) {
    const float et = ex2_approx(__fmul_rn(__fsub_rn(xt, rn.mt), c));
    if (!RESID) return et;
    const float ed = ex2_approx(__fmul_rn(__fsub_rn(xd, rn.md), c));
    return fmaxf(__fmaf_rn(-ed, rn.rho_lo, __fmaf_rn(-ed, rn.rho_hi, et)), 0.0f);
}

__device__ __forceinline__ double warp_inclusive_scan(double v, int lane) {
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    return v;
}

// One position of Sec. 3.2 (steps 1-5) with the guards of Sec. 3.3 item 2, in fp64:
// P_t(x), P_d(x) from the token's logits and the rows' (max, Z); max P_t = 1/Z_t (the largest
// term of Z is exp(0)); R = P_t(x) / max(P_d(x), eps); Tolerance = beta (1 - max P_t);
// accept iff R >= max(U - Tolerance, 0).  cls: 0 reject, 1 direct accept (R >= U), 2 pardon.
struct Decision { double pt, pd, maxp; int cls; bool accept; };

__device__ __forceinline__ Decision decide_position(double lt, double ld, float2 st, float2 sd, double T,
                                                    double beta, double U) {
    Decision r;
    r.pt = exp((lt - (double)st.x) / T) / (double)st.y;
    r.pd = exp((ld - (double)sd.x) / T) / (double)sd.y;
    r.maxp = 1.0 / (double)st.y;
    const double ratio = r.pt / fmax(r.pd, kEps);
    const double tol = beta * (1.0 - r.maxp);
    const double thr = fmax(U - tol, 0.0);
    r.accept = ratio >= thr;
    r.cls = ratio >= U ? 1 : (r.accept ? 2 : 0);
    return r;
}

// (m, Z) of a row is usable when the maximum is finite and the sum positive and finite (NaN fails).
__device__ __forceinline__ bool rowstat_ok(float m, float s) {
    return m > -INFINITY && m < INFINITY && s > 0.0f && s < INFINITY;
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint32_t max_f16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// ---- statistics of a slice ------------------------------------------------------
// Running (m, s) of one thread: s = sum exp2(fl(l c - mu)), mu = fl(m c) (0 while m = -inf).
// One fused multiply-add per entry; the rounding of m c is taken out again in acc_close.
struct RowAcc { float m, mu, s[4]; };

__device__ __forceinline__ void acc_open(RowAcc& a) { a.m = -INFINITY; a.mu = 0.f; a.s[0] = a.s[1] = a.s[2] = a.s[3] = 0.f; }

__device__ __forceinline__ void acc_raise(RowAcc& a, float cm, float c) {
    if (cm > a.m) {  // false for NaN: a NaN entry reaches the sum instead
        const float mu_new = cm * c;
        const float sc = (a.m == -INFINITY) ? 0.f : ex2_approx(a.mu - mu_new);
        a.s[0] *= sc; a.s[1] *= sc; a.s[2] *= sc; a.s[3] *= sc;
        a.m = cm;
        a.mu = mu_new;
    }
}

// -> (m, s) with s relative to the exact product m c: fl(m c) differs from m c by
// delta = fma(m, c, -fl(m c)) exactly; the terms were taken relative to fl(m c) = m c - delta, so
// every one carries the factor 2^delta, which is divided out: 2^-delta = 1 - delta ln 2 to first
// order (|delta| < 1e-5).
__device__ __forceinline__ float2 acc_close(const RowAcc& a, float c) {
    float s = (a.s[0] + a.s[1]) + (a.s[2] + a.s[3]);
    if (a.m > -INFINITY && a.m < INFINITY) s = __fmaf_rn(s, -0.6931471805599453f * __fmaf_rn(a.m, c, -a.mu), s);
    return make_float2(a.m, s);
}

// s, a sum of exp2((l - m) c), expressed relative to the maximum M >= m instead.  An empty part
// (m = -inf) contributes nothing; NaN sums stay NaN.
__device__ __forceinline__ float rebase_sum(float m, float s, float M, float c) {
    const float sc = (m == -INFINITY) ? 0.f : exp2f((m - M) * c);   // full precision: the factor scales a whole part
    return s * sc;
}

template <typename E> struct SubLoad;
template <> struct SubLoad<float> {
    // two 16-byte vectors of a full sub-chunk and their maximum
    __device__ static __forceinline__ float load(const unsigned char* buf, int v0, int v1, float (&x)[2][4]) {
        Vec<float>::load(buf, v0, x[0]);
        Vec<float>::load(buf, v1, x[1]);
        return fmaxf(fmaxf(fmaxf(x[0][0], x[0][1]), fmaxf(x[0][2], x[0][3])),
                     fmaxf(fmaxf(x[1][0], x[1][1]), fmaxf(x[1][2], x[1][3])));
    }
};
template <> struct SubLoad<uint16_t> {
    __device__ static __forceinline__ float load(const unsigned char* buf, int v0, int v1, float (&x)[2][8]) {
        const uint4 a = reinterpret_cast<const uint4*>(buf)[v0];
        const uint4 b = reinterpret_cast<const uint4*>(buf)[v1];
        // the maximum of bf16 pairs is exact in packed form: half an instruction per entry
        const uint32_t pm = max_bf16x2(max_bf16x2(max_bf16x2(a.x, a.y), max_bf16x2(a.z, a.w)),
                                       max_bf16x2(max_bf16x2(b.x, b.y), max_bf16x2(b.z, b.w)));
        x[0][0] = __uint_as_float(a.x << 16); x[0][1] = __uint_as_float(a.x & 0xffff0000u);
        x[0][2] = __uint_as_float(a.y << 16); x[0][3] = __uint_as_float(a.y & 0xffff0000u);
        x[0][4] = __uint_as_float(a.z << 16); x[0][5] = __uint_as_float(a.z & 0xffff0000u);
        x[0][6] = __uint_as_float(a.w << 16); x[0][7] = __uint_as_float(a.w & 0xffff0000u);
        x[1][0] = __uint_as_float(b.x << 16); x[1][1] = __uint_as_float(b.x & 0xffff0000u);
        x[1][2] = __uint_as_float(b.y << 16); x[1][3] = __uint_as_float(b.y & 0xffff0000u);
        x[1][4] = __uint_as_float(b.z << 16); x[1][5] = __uint_as_float(b.z & 0xffff0000u);
        x[1][6] = __uint_as_float(b.w << 16); x[1][7] = __uint_as_float(b.w & 0xffff0000u);
        return fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xffff0000u));
    }
};
template <> struct SubLoad<f16_t> {
    __device__ static __forceinline__ float load(const unsigned char* buf, int v0, int v1, float (&x)[2][8]) {
        const uint4 a = reinterpret_cast<const uint4*>(buf)[v0];
        const uint4 b = reinterpret_cast<const uint4*>(buf)[v1];
        const uint32_t pm = max_f16x2(max_f16x2(max_f16x2(a.x, a.y), max_f16x2(a.z, a.w)),
                                      max_f16x2(max_f16x2(b.x, b.y), max_f16x2(b.z, b.w)));
        Vec<f16_t>::unpack(a, x[0]);
        Vec<f16_t>::unpack(b, x[1]);
        const float2 m = f16x2_to_float2(pm);
        return fmaxf(m.x, m.y);
    }
};

// Two 16-byte vectors (indices v0, v1) of a staged row piece holding n valid entries from its
// start; `full` says that both vectors lie wholly inside the piece.
template <typename E>
__device__ __forceinline__ void stats_two_vectors(const unsigned char* buf, int v0, int v1, bool full, int n, float c, RowAcc& a) {
    constexpr int N = Vec<E>::N;
    float x[2][N];
    float cm;
    if (full) {
        cm = SubLoad<E>::load(buf, v0, v1, x);
    } else {  // ragged end: what lies beyond the piece counts as -inf
        Vec<E>::load(buf, v0, x[0]);
        Vec<E>::load(buf, v1, x[1]);
        cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            if (v0 * N + i >= n) x[0][i] = -INFINITY;
            if (v1 * N + i >= n) x[1][i] = -INFINITY;
            cm = fmaxf(cm, fmaxf(x[0][i], x[1][i]));
        }
    }
    acc_raise(a, cm, c);
    const float nmu = -a.mu;
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) a.s[i & 3] += ex2_approx(__fmaf_rn(x[j][i], c, nmu));
}

}  // namespace ears
