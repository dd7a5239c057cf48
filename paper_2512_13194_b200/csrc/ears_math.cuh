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
//
// The uncertainty that scales the tolerance is 1 - max P_t as printed (Sec. 3.2), or -- when the
// caller asks for it and passes unc >= 0 -- the normalised entropy H(P_t) / ln V (Sec. 5 names the
// entropy as a more refined measure; the normalisation is this library's reading).
struct Decision { double pt, pd, maxp; int cls; bool accept; };

__device__ __forceinline__ Decision decide_position(double lt, double ld, float2 st, float2 sd, double T,
                                                    double beta, double U, double unc = -1.0) {
    Decision r;
    r.pt = exp((lt - (double)st.x) / T) / (double)st.y;
    r.pd = exp((ld - (double)sd.x) / T) / (double)sd.y;
    r.maxp = 1.0 / (double)st.y;
    const double ratio = r.pt / fmax(r.pd, kEps);
    const double tol = beta * (unc >= 0.0 ? unc : 1.0 - r.maxp);
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

// ---- two fp32 lanes per instruction ---------------------------------------------
// sm_100 issues fused multiply-adds, additions and multiplications on pairs of fp32 values held in
// a 64-bit register (fma.rn.f32x2 and friends): the same roundings as the scalar forms, half the
// issue slots.  The streaming loops spend one multiply-add and one addition per logit, so this is
// where their instruction count comes from.
typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// exp2 of both lanes (the special-function unit has no paired form)
__device__ __forceinline__ f32x2 ex2_pair(f32x2 v) {
    float lo, hi;
    unpack2(v, lo, hi);
    return pack2(ex2_approx(lo), ex2_approx(hi));
}
// the largest of three (sm_100 takes three operands in one instruction); a NaN operand is
// ignored, like fmaxf does
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// ---- statistics of a slice ------------------------------------------------------
// Running (m, s) of one thread: s = sum exp2(fl(l c - mu)), mu = fl(m c) (0 while m = -inf).
// One fused multiply-add per entry; the rounding of m c is taken out again in acc_close.
// The sum is kept in four lanes (two register pairs) so that consecutive additions overlap.
//
// ENT: the entropy of the row comes out of the same sweep.  With t = l c - mu (log2 units below
// the reference) and e = 2^t, the thread also carries w = sum e t (one more multiply-add per
// entry): H = ln Z - ln 2 * (sum e t) / Z.  Every t is <= 0 up to rounding, so nothing cancels.
// Masked entries (l = -inf) would give 0 * -inf; the ENT loops therefore read their logits through
// a clamp at a large negative finite value (NaNs pass the clamp and still reach the sums).
template <bool ENT> struct RowAccT { float m, mu; f32x2 s[2]; f32x2 w[ENT ? 2 : 1]; };
typedef RowAccT<false> RowAcc;

constexpr float kLogitFloor = -1.0e30f;   // what -inf logits are read as where products with them must stay finite

template <bool ENT>
__device__ __forceinline__ void acc_open(RowAccT<ENT>& a) {
    a.m = -INFINITY; a.mu = 0.f; a.s[0] = a.s[1] = pack2(0.f, 0.f);
    if (ENT) a.w[0] = a.w[ENT ? 1 : 0] = pack2(0.f, 0.f);
}

template <bool ENT>
__device__ __forceinline__ void acc_raise(RowAccT<ENT>& a, float cm, float c) {
    if (cm > a.m) {  // false for NaN: a NaN entry reaches the sum instead
        const float mu_new = cm * c;
        const float sc = (a.m == -INFINITY) ? 0.f : ex2_approx(a.mu - mu_new);
        const f32x2 sc2 = pack2(sc, sc);
        if (ENT) {
            // every t drops by mu_new - mu and every e shrinks by sc: w <- sc (w - (mu_new - mu) s)
            const float dl = (a.m == -INFINITY) ? 0.f : a.mu - mu_new;
            const f32x2 dl2 = pack2(dl, dl);
            a.w[0] = mul2(fma2(dl2, a.s[0], a.w[0]), sc2);
            a.w[ENT ? 1 : 0] = mul2(fma2(dl2, a.s[1], a.w[ENT ? 1 : 0]), sc2);
        }
        a.s[0] = mul2(a.s[0], sc2);
        a.s[1] = mul2(a.s[1], sc2);
        a.m = cm;
        a.mu = mu_new;
    }
}

// One more entry (loops that go element by element: rows that are not 16-byte aligned).
template <bool ENT>
__device__ __forceinline__ void acc_add_one(RowAccT<ENT>& a, float x, float c) {
    if (ENT) x = fmaxf(x, kLogitFloor) + (x != x ? x : 0.f);   // -inf -> floor; NaN stays NaN
    const float t = __fmaf_rn(x, c, -a.mu), e = ex2_approx(t);
    a.s[0] = add2(a.s[0], pack2(e, 0.f));
    if (ENT) a.w[0] = add2(a.w[0], pack2(e * t, 0.f));
}

// Two more pairs of entries: sum += exp2(x c - mu) in each of the four lanes.
template <bool ENT>
__device__ __forceinline__ void acc_add_pairs(RowAccT<ENT>& a, f32x2 x01, f32x2 x23, f32x2 c2, f32x2 nmu2) {
    const f32x2 t0 = fma2(x01, c2, nmu2), t1 = fma2(x23, c2, nmu2);
    const f32x2 e0 = ex2_pair(t0), e1 = ex2_pair(t1);
    a.s[0] = add2(a.s[0], e0);
    a.s[1] = add2(a.s[1], e1);
    if (ENT) {
        a.w[0] = fma2(e0, t0, a.w[0]);
        a.w[ENT ? 1 : 0] = fma2(e1, t1, a.w[ENT ? 1 : 0]);
    }
}

// -> (m, s) with s relative to the exact product m c: fl(m c) differs from m c by
// delta = fma(m, c, -fl(m c)) exactly; the terms were taken relative to fl(m c) = m c - delta, so
// every one carries the factor 2^delta, which is divided out: 2^-delta = 1 - delta ln 2 to first
// order (|delta| < 1e-5).
// ENT: *w_out = sum e t relative to the exact product as well: the terms used t + delta and
// e 2^delta, so w_used = 2^delta (w + delta s); both effects are taken out to first order.
template <bool ENT>
__device__ __forceinline__ float2 acc_close(const RowAccT<ENT>& a, float c, float* w_out = nullptr) {
    float s0, s1;
    unpack2(add2(a.s[0], a.s[1]), s0, s1);
    float s = s0 + s1, w = 0.f;
    if (ENT) {
        float w0, w1;
        unpack2(add2(a.w[0], a.w[ENT ? 1 : 0]), w0, w1);
        w = w0 + w1;
    }
    if (a.m > -INFINITY && a.m < INFINITY) {
        const float delta = __fmaf_rn(a.m, c, -a.mu);
        const float k = -0.6931471805599453f * delta;
        s = __fmaf_rn(s, k, s);
        if (ENT) w = __fmaf_rn(-delta, s, __fmaf_rn(w, k, w));
    }
    if (ENT && w_out) *w_out = w;
    return make_float2(a.m, s);
}

// s, a sum of exp2((l - m) c), expressed relative to the maximum M >= m instead.  An empty part
// (m = -inf) contributes nothing; NaN sums stay NaN.
__device__ __forceinline__ float rebase_sum(float m, float s, float M, float c) {
    const float sc = (m == -INFINITY) ? 0.f : exp2f((m - M) * c);   // full precision: the factor scales a whole part
    return s * sc;
}

// The same for the pair (s, w = sum e t): relative to M every t is lower by (M - m) c.
__device__ __forceinline__ float2 rebase_sum_w(float m, float s, float w, float M, float c) {
    if (m == -INFINITY) return make_float2(s * 0.f, 0.f);
    const float dl = (m - M) * c;
    const float sc = exp2f(dl);
    return make_float2(s * sc, sc * __fmaf_rn(dl, s, w));
}

// Entropy (nats) of a row from Z = sum e and w = sum e t (t in log2 units below the row maximum):
// ln p = t ln 2 - ln Z, hence H = ln Z - ln 2 * w / Z.  fp64: called once per position.
__device__ __forceinline__ double row_entropy(float Z, float w) {
    return log((double)Z) - 0.6931471805599453 * (double)w / (double)Z;
}
// H / ln V, the uncertainty in [0, 1] that the entropy gives (0 for a vocabulary of one entry).
__device__ __forceinline__ double entropy_uncertainty(double H, int V) {
    return V > 1 ? fmin(fmax(H / log((double)V), 0.0), 1.0) : 0.0;
}

// larger of two, a NaN operand wins (so that a clamp from below lets NaNs through)
__device__ __forceinline__ float max_nan(float a, float b) {
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t max_nan_f16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.NaN.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// ---- packed 16-byte vectors of logits ---------------------------------------------
// A vector stays packed (four 32-bit words, as loaded) until it is used.  Per element type:
//   N            entries per vector
//   vmax_all     the largest entry of G vectors (on packed pairs for the 2-byte types, which is exact;
//                three operands per instruction for fp32); NaN entries are ignored here and reach the
//                sum instead
//   pairs        the entries widened to fp32, two per 64-bit register
//   unpack       the entries widened to fp32, one per register
//   floor_inf    the vector with its -inf entries raised to a large negative finite value (NaNs stay)
//   minus_inf    a vector of -inf entries;  mask_tail: entries from index `keep` on become -inf
//   gather       up to N entries fetched one by one (rows that are not 16-byte aligned)
template <typename E> struct Words;
template <> struct Words<float> {
    static constexpr int N = 4;
    template <int G>
    __device__ static __forceinline__ float vmax_all(const uint4 (&w)[G]) {
        float cm = max3(__uint_as_float(w[0].x), __uint_as_float(w[0].y), __uint_as_float(w[0].z));
        cm = fmaxf(cm, __uint_as_float(w[0].w));
#pragma unroll
        for (int j = 1; j < G; ++j) {
            cm = max3(cm, __uint_as_float(w[j].x), __uint_as_float(w[j].y));
            cm = max3(cm, __uint_as_float(w[j].z), __uint_as_float(w[j].w));
        }
        return cm;
    }
    __device__ static __forceinline__ void pairs(uint4 w, f32x2 (&p)[2]) {
        p[0] = pack2(__uint_as_float(w.x), __uint_as_float(w.y));
        p[1] = pack2(__uint_as_float(w.z), __uint_as_float(w.w));
    }
    __device__ static __forceinline__ void unpack(uint4 w, float (&x)[4]) {
        x[0] = __uint_as_float(w.x); x[1] = __uint_as_float(w.y); x[2] = __uint_as_float(w.z); x[3] = __uint_as_float(w.w);
    }
    __device__ static __forceinline__ uint4 floor_inf(uint4 w) {
        return make_uint4(__float_as_uint(max_nan(__uint_as_float(w.x), kLogitFloor)), __float_as_uint(max_nan(__uint_as_float(w.y), kLogitFloor)),
                          __float_as_uint(max_nan(__uint_as_float(w.z), kLogitFloor)), __float_as_uint(max_nan(__uint_as_float(w.w), kLogitFloor)));
    }
    __device__ static __forceinline__ uint4 minus_inf() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    __device__ static __forceinline__ uint4 mask_tail(uint4 w, int keep) {
        if (keep < 1) w.x = 0xff800000u;
        if (keep < 2) w.y = 0xff800000u;
        if (keep < 3) w.z = 0xff800000u;
        if (keep < 4) w.w = 0xff800000u;
        return w;
    }
    // up to N entries from p (fewer, or none, when `left` says so), the rest -inf
    __device__ static __forceinline__ uint4 gather(const float* p, int left) {
        uint4 w = minus_inf();
        if (left > 0) w.x = __float_as_uint(__ldg(p));
        if (left > 1) w.y = __float_as_uint(__ldg(p + 1));
        if (left > 2) w.z = __float_as_uint(__ldg(p + 2));
        if (left > 3) w.w = __float_as_uint(__ldg(p + 3));
        return w;
    }
};
// entries from `keep` on of a vector of eight 2-byte entries become `ninf` (the type's -inf pattern)
__device__ __forceinline__ uint4 mask_tail16(uint4 w, int keep, uint32_t ninf) {
    uint32_t h[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (keep <= 2 * i) h[i] = ninf | (ninf << 16);
        else if (keep == 2 * i + 1) h[i] = (h[i] & 0xffffu) | (ninf << 16);
    }
    return make_uint4(h[0], h[1], h[2], h[3]);
}
template <> struct Words<uint16_t> {
    static constexpr int N = 8;
    template <int G>
    __device__ static __forceinline__ float vmax_all(const uint4 (&w)[G]) {   // exact on packed pairs
        uint32_t pm = max_bf16x2(max_bf16x2(w[0].x, w[0].y), max_bf16x2(w[0].z, w[0].w));
#pragma unroll
        for (int j = 1; j < G; ++j) pm = max_bf16x2(max_bf16x2(pm, w[j].x), max_bf16x2(max_bf16x2(w[j].y, w[j].z), w[j].w));
        return fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xffff0000u));
    }
    __device__ static __forceinline__ f32x2 widen(uint32_t h) { return pack2(__uint_as_float(h << 16), __uint_as_float(h & 0xffff0000u)); }
    __device__ static __forceinline__ void pairs(uint4 w, f32x2 (&p)[4]) {
        p[0] = widen(w.x); p[1] = widen(w.y); p[2] = widen(w.z); p[3] = widen(w.w);
    }
    __device__ static __forceinline__ void unpack(uint4 w, float (&x)[8]) {
        x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xffff0000u);
        x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xffff0000u);
        x[4] = __uint_as_float(w.z << 16); x[5] = __uint_as_float(w.z & 0xffff0000u);
        x[6] = __uint_as_float(w.w << 16); x[7] = __uint_as_float(w.w & 0xffff0000u);
    }
    __device__ static __forceinline__ uint4 floor_inf(uint4 w) {   // 0xf149: about -1e30 as bfloat16
        return make_uint4(max_nan_bf16x2(w.x, 0xf149f149u), max_nan_bf16x2(w.y, 0xf149f149u), max_nan_bf16x2(w.z, 0xf149f149u),
                          max_nan_bf16x2(w.w, 0xf149f149u));
    }
    __device__ static __forceinline__ uint4 minus_inf() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
    __device__ static __forceinline__ uint4 mask_tail(uint4 w, int keep) { return mask_tail16(w, keep, 0xff80u); }
    __device__ static __forceinline__ uint4 gather(const uint16_t* p, int left) {
        uint32_t h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = i < left ? (uint32_t)__ldg(p + i) : 0xff80u;
        return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
    }
};
template <> struct Words<f16_t> {
    static constexpr int N = 8;
    template <int G>
    __device__ static __forceinline__ float vmax_all(const uint4 (&w)[G]) {   // exact on packed pairs
        uint32_t pm = max_f16x2(max_f16x2(w[0].x, w[0].y), max_f16x2(w[0].z, w[0].w));
#pragma unroll
        for (int j = 1; j < G; ++j) pm = max_f16x2(max_f16x2(pm, w[j].x), max_f16x2(max_f16x2(w[j].y, w[j].z), w[j].w));
        const float2 m = f16x2_to_float2(pm);
        return fmaxf(m.x, m.y);
    }
    __device__ static __forceinline__ f32x2 widen(uint32_t h) { const float2 v = f16x2_to_float2(h); return pack2(v.x, v.y); }
    __device__ static __forceinline__ void pairs(uint4 w, f32x2 (&p)[4]) {
        p[0] = widen(w.x); p[1] = widen(w.y); p[2] = widen(w.z); p[3] = widen(w.w);
    }
    __device__ static __forceinline__ void unpack(uint4 w, float (&x)[8]) { Vec<f16_t>::unpack(w, x); }
    __device__ static __forceinline__ uint4 floor_inf(uint4 w) {   // 0xfbff: -65504, the lowest finite binary16
        return make_uint4(max_nan_f16x2(w.x, 0xfbfffbffu), max_nan_f16x2(w.y, 0xfbfffbffu), max_nan_f16x2(w.z, 0xfbfffbffu),
                          max_nan_f16x2(w.w, 0xfbfffbffu));
    }
    __device__ static __forceinline__ uint4 minus_inf() { return make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u); }
    __device__ static __forceinline__ uint4 mask_tail(uint4 w, int keep) { return mask_tail16(w, keep, 0xfc00u); }
    __device__ static __forceinline__ uint4 gather(const f16_t* p, int left) {
        uint32_t h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = i < left ? (uint32_t)__ldg(&p[i].bits) : 0xfc00u;
        return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
    }
};

// G vectors of one thread: maximum first, one rescale of the running sums if it grew, then one
// multiply-add, one exp2 and one addition per entry, the first and the last on pairs.
template <typename E, int G, bool ENT>
__device__ __forceinline__ void fold_vectors(const uint4 (&w)[G], float c, RowAccT<ENT>& a) {
    constexpr int PN = Words<E>::N / 2;
    acc_raise(a, Words<E>::template vmax_all<G>(w), c);
    const f32x2 c2 = pack2(c, c), nmu2 = pack2(-a.mu, -a.mu);
#pragma unroll
    for (int j = 0; j < G; ++j) {
        f32x2 p[PN];
        Words<E>::pairs(ENT ? Words<E>::floor_inf(w[j]) : w[j], p);
#pragma unroll
        for (int i = 0; i < PN; i += 2) acc_add_pairs(a, p[i], p[i + 1], c2, nmu2);
    }
}

// Two 16-byte vectors (indices v0, v1) of a staged row piece holding n valid entries from its
// start; `full` says that both vectors lie wholly inside the piece.
template <typename E, bool ENT>
__device__ __forceinline__ void stats_two_vectors(const unsigned char* buf, int v0, int v1, bool full, int n, float c, RowAccT<ENT>& a) {
    constexpr int N = Words<E>::N;
    uint4 w[2] = {reinterpret_cast<const uint4*>(buf)[v0], reinterpret_cast<const uint4*>(buf)[v1]};
    if (!full) {  // ragged end: what lies beyond the piece counts as -inf
        w[0] = Words<E>::mask_tail(w[0], n - v0 * N);
        w[1] = Words<E>::mask_tail(w[1], n - v1 * N);
    }
    fold_vectors<E, 2, ENT>(w, c, a);
}

}  // namespace ears
