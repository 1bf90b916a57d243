// Device-side building blocks of the PPOW scoring pass (sm_100a).
//
// A logit row is reduced in log2 units against a *stale reference*: with s = log2(e)/T,
//   x_a(v) = a_v*s - rho_a,   x_b(v) = b_v*s - rho_b
// where rho_a / rho_b are per-thread references that are only raised when a tile's maximum
// exceeds them by more than REBASE_LOG2, so no per-element rescale is needed.  The threshold is
// small on purpose: x is rounded to f32, so a term 2^x carries a relative error of 0.5*ulp(x)*ln2,
// and a confident distribution has ONE term that decides the sum.  Keeping every x <= 4 bounds
// that error at 1.7e-7; terms far below the reference are many and their errors average out.
// Each thread accumulates
//   Sa = sum 2^x_a     Sb = sum 2^x_b     E = sum 2^x_a * x_a     D = sum 2^x_a * (x_a - x_b)
// from which (Sec. 4.2)  H(P)/ln2 = log2 Sa - E/Sa  and  KL(P||Q)/ln2 = D/Sa - log2 Sa + log2 Sb.
// When the reverse divergence of the training objective is wanted (Sec. 4.1, App. A.2) one more sum,
//   B = sum 2^x_b * (x_a - x_b),   gives   KL(Q||P)/ln2 = -B/Sb - log2 Sb + log2 Sa.
// Accumulating D from the per-element difference (not E - F) avoids cancelling two O(10) terms
// to reach a KL of O(0.01).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ppow {

// Storage tags of 16-bit logits: uint16_t stands for bf16 bit patterns, half_bits for IEEE binary16.
struct half_bits {
    uint16_t bits;
};
__device__ __forceinline__ float f16_to_f32(uint16_t bits) { return __half2float(__ushort_as_half(bits)); }

constexpr float REBASE_LOG2 = 4.0f;      // raise a reference when a tile exceeds it by 2^4
constexpr float RHO_INIT = -1.0e30f;     // "no reference yet": the first tile always rebases

// References are whole numbers (log2 units), so moving a sum from one reference to another multiplies it by an
// exact power of two: no rounding in rebase(), none when partial sums of a row are merged.
// 2^d for a whole number d <= 0 (0 below the normal range: the sum it scales is negligible there).
__device__ __forceinline__ float pow2_whole(float d)
{
    return d < -126.0f ? 0.0f : __int_as_float((127 + (int)d) << 23);
}
__device__ __forceinline__ double pow2_whole(double d)
{
    return d < -1022.0 ? 0.0 : __longlong_as_double((long long)(1023 + (int)d) << 52);
}

// One partial reduction of (part of) a row; merged later in float64.
struct __align__(16) RowPartial {
    float rho_a, rho_b;   // references, log2 units
    double Sa, Sb;        // sums relative to those references
    double E, D;          // weighted sums relative to the same references
    double B;             // sum 2^x_b (x_a - x_b), for KL(Q||P); 0 unless the call asks for it
    float max_a;          // largest stored target logit seen
    int32_t argmax;       // its lowest vocabulary index
};
static_assert(sizeof(RowPartial) == 64, "RowPartial layout");

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Per-thread running state for one row (or row segment).
//
// A confident distribution puts almost all of a sum into one term: once an f32 accumulator holds
// that term, every later small term is rounded at its ulp (6e-8 relative each, thousands of times
// when a lane walks a whole row).  So all sums are kept as tile-local partials (Sa, Sb, E, D, restarted
// from zero by flush()), and only the few adds inside one tile can be absorbed.  Sa and Sb, which the
// log-probabilities are read from, are folded into running (hi, lo) pairs with an error-compensated
// add; for the weighted sums E, D (and B) a plain add per tile measures the same against the float64
// definition (their tolerance is relative to an entropy or a divergence, not to a log-probability).
//
// The tile-local accumulators are float2: lane .x takes the even vocabulary entries of a packed bf16
// word, lane .y the odd ones, so that the arithmetic runs on sm_100's packed f32x2 instructions
// (__ffma2_rn / __fadd2_rn: one issue slot for two IEEE fma/add operations).
// REV: also accumulate B for KL(Q||P) (one more packed fma per word; members unused otherwise).
template <bool REV>
struct RowAcc {
    float rho_a, rho_b;
    float2 Sa, Sb, E, D, B;
    float Sa_hi, Sa_lo, Sb_hi, Sb_lo;   // compensated running sums of 2^x
    float Et, Dt, Bt;                   // running weighted sums
    float max_a;
    int32_t best;       // where max_a was first seen (meaning defined by the caller)

    __device__ __forceinline__ void reset()
    {
        rho_a = rho_b = RHO_INIT;
        Sa = Sb = E = D = B = make_float2(0.0f, 0.0f);
        Sa_hi = Sa_lo = Sb_hi = Sb_lo = Et = Dt = Bt = 0.0f;
        max_a = -INFINITY;
        best = 0;
    }

    // hi + p -> (hi, lo += rounding error); p and hi of any sign (Knuth's two-sum).
    static __device__ __forceinline__ void two_sum(float &hi, float &lo, float p)
    {
        const float t = hi + p;
        const float bp = t - hi;
        lo += (hi - (t - bp)) + (p - bp);
        hi = t;
    }

    // Fold the tile-local partial sums into the compensated running sums (call once per tile).
    __device__ __forceinline__ void flush()
    {
        two_sum(Sa_hi, Sa_lo, Sa.x + Sa.y);
        two_sum(Sb_hi, Sb_lo, Sb.x + Sb.y);
        Et += E.x + E.y;   // see the note on the struct: a plain add is enough for these three
        Dt += D.x + D.y;
        if (REV) Bt += B.x + B.y;
        Sa = Sb = E = D = B = make_float2(0.0f, 0.0f);
    }

    // Move both references (log2 units).  Only between tiles (after flush()).  With x' = x - d,
    //   Sa' = fa*Sa,  E' = fa*(E + da*Sa),  D' = fa*(D + (da - db)*Sa),  Sb' = fb*Sb,  B' = fb*(B + (da - db)*Sb)
    // where da = rho_a - new_rho_a <= 0 and fa = 2^da (same for b).  Applying (da - db) in one step
    // keeps D exactly 0 when draft and target are the same data.
    __device__ __forceinline__ void rebase(float new_rho_a, float new_rho_b)
    {
        const float da = rho_a - new_rho_a, db = rho_b - new_rho_b;
        if (da == 0.0f && db == 0.0f) return;
        const float fa = pow2_whole(da), fb = pow2_whole(db);   // exact: references are whole numbers
        const float S = Sa_hi + Sa_lo;
        Et = fa * fmaf(da, S, Et);
        Dt = fa * fmaf(da - db, S, Dt);
        if (REV) Bt = fb * fmaf(da - db, Sb_hi + Sb_lo, Bt);
        Sa_hi *= fa;
        Sa_lo *= fa;
        Sb_hi *= fb;
        Sb_lo *= fb;
        rho_a = new_rho_a;
        rho_b = new_rho_b;
    }

    // One (target, draft) pair already widened to f32 (scalar path; accumulates into lane .x).
    __device__ __forceinline__ void add_pair(float a, float b, float s)
    {
        const float xa = fmaf(a, s, -rho_a);
        const float xb = fmaf(b, s, -rho_b);
        const float ea = ex2_approx(xa);
        const float eb = ex2_approx(xb);
        Sa.x += ea;
        Sb.x += eb;
        E.x = fmaf(ea, xa, E.x);
        D.x = fmaf(ea, xa - xb, D.x);
        if (REV) B.x = fmaf(eb, xa - xb, B.x);
    }

    // Two pairs at once: the same operations as two add_pair calls, on packed f32x2 instructions.
    // a = two target logits, b = the two draft logits at the same vocabulary entries;
    // s2 = (s, s), nra = (-rho_a, -rho_a), nrb = (-rho_b, -rho_b).
    __device__ __forceinline__ void add2(float2 a, float2 b, float2 s2, float2 nra, float2 nrb)
    {
        const float2 xa = __ffma2_rn(a, s2, nra);
        const float2 xb = __ffma2_rn(b, s2, nrb);
        const float2 ea = make_float2(ex2_approx(xa.x), ex2_approx(xa.y));
        const float2 eb = make_float2(ex2_approx(xb.x), ex2_approx(xb.y));
        Sa = __fadd2_rn(Sa, ea);
        Sb = __fadd2_rn(Sb, eb);
        E = __ffma2_rn(ea, xa, E);
        const float2 dx = __ffma2_rn(xb, make_float2(-1.0f, -1.0f), xa);   // xa - xb, one rounding
        D = __ffma2_rn(ea, dx, D);
        if (REV) B = __ffma2_rn(eb, dx, B);
    }

    // One packed bf16 word of each tensor (even entry in the low half).
    __device__ __forceinline__ void add_word(uint32_t wa, uint32_t wb, float2 s2, float2 nra, float2 nrb)
    {
        add2(make_float2(bf16_lo(wa), bf16_hi(wa)), make_float2(bf16_lo(wb), bf16_hi(wb)), s2, nra, nrb);
    }

    // Raise the references if this tile's maxima (raw logit units) call for it.
    __device__ __forceinline__ void guard(float tile_max_a, float tile_max_b, float s)
    {
        const bool up_a = fmaf(tile_max_a, s, -rho_a) > REBASE_LOG2;
        const bool up_b = fmaf(tile_max_b, s, -rho_b) > REBASE_LOG2;
        if (up_a | up_b) rebase(up_a ? ceilf(tile_max_a * s) : rho_a, up_b ? ceilf(tile_max_b * s) : rho_b);
    }
};

// ---- storage formats: one 16-byte unit of logits, and one logit at a time ---------------------------
// mask_unit: the logits of a unit outside [lo, hi) do not belong to the row being read (a row that starts or
// ends inside a unit); they are replaced by a finite, hugely negative value (-1e25, -65504 in binary16): its
// term 2^x is 0 and 0 * x stays 0, which -inf would not.

__device__ __forceinline__ void mask_halves(uint4 &w4, int lo, int hi, uint32_t bits)
{
    uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (2 * q < lo || 2 * q >= hi) w[q] = (w[q] & 0xffff0000u) | bits;
        if (2 * q + 1 < lo || 2 * q + 1 >= hi) w[q] = (w[q] & 0x0000ffffu) | (bits << 16);
    }
    w4 = make_uint4(w[0], w[1], w[2], w[3]);
}

struct UnitBf16 {
    static constexpr int EPU = 8;   // logits per unit
    static __device__ __forceinline__ uint4 none() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
    static __device__ __forceinline__ float unit_max(const uint4 &w)
    {
        const uint32_t m = max_bf16x2(max_bf16x2(w.x, w.y), max_bf16x2(w.z, w.w));
        return fmaxf(bf16_lo(m), bf16_hi(m));
    }
    static __device__ __forceinline__ void unpack(const uint4 &w, float (&f)[8])
    {
        f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
        f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w, int lo, int hi) { mask_halves(w, lo, hi, 0xe904u); }
};

struct UnitF16 {
    static constexpr int EPU = 8;
    static __device__ __forceinline__ uint4 none() { return make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u); }
    static __device__ __forceinline__ __half2 h2(uint32_t w) { return *reinterpret_cast<const __half2 *>(&w); }
    static __device__ __forceinline__ float unit_max(const uint4 &w)
    {
        const float2 f = __half22float2(__hmax2(__hmax2(h2(w.x), h2(w.y)), __hmax2(h2(w.z), h2(w.w))));
        return fmaxf(f.x, f.y);
    }
    static __device__ __forceinline__ void unpack(const uint4 &w, float (&f)[8])
    {
        const float2 a = __half22float2(h2(w.x)), b = __half22float2(h2(w.y));
        const float2 c = __half22float2(h2(w.z)), d = __half22float2(h2(w.w));
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w, int lo, int hi) { mask_halves(w, lo, hi, 0xfbffu); }
};

struct UnitF32 {
    static constexpr int EPU = 4;
    static __device__ __forceinline__ uint4 none() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    static __device__ __forceinline__ float unit_max(const uint4 &w)
    {
        return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)), fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
    }
    static __device__ __forceinline__ void unpack(const uint4 &w, float (&f)[4])
    {
        f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y); f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w, int lo, int hi)
    {
        const uint32_t m = 0xe9045951u;   // -1e25
        if (0 < lo || 0 >= hi) w.x = m;
        if (1 < lo || 1 >= hi) w.y = m;
        if (2 < lo || 2 >= hi) w.z = m;
        if (3 < lo || 3 >= hi) w.w = m;
    }
};

// A row of V logits that may start inside a 16-byte unit (SHIFTED; otherwise rows are whole aligned units and
// nothing is masked): where its units begin, how many it spans, and which logits of unit `ui` belong to it.
template <typename Unit, bool SHIFTED>
struct RowSpan {
    const uint4 *base;     // aligned address of the unit that holds the row's first logit
    int32_t head, span, units;   // logits of unit 0 before the row; head + V; units the row touches
    __device__ __forceinline__ RowSpan(const void *tensor, size_t row, int32_t V)
    {
        constexpr int ES = 16 / Unit::EPU;
        const uintptr_t a = reinterpret_cast<uintptr_t>(tensor) + row * (size_t)V * ES;
        base = reinterpret_cast<const uint4 *>(a & ~(uintptr_t)15);
        head = SHIFTED ? (int32_t)((a & 15u) / ES) : 0;
        span = head + V;
        units = (span + Unit::EPU - 1) / Unit::EPU;
    }
    __device__ __forceinline__ bool touches(int32_t ui) const { return ui == 0 || ui == units - 1; }
    __device__ __forceinline__ void mask(uint4 &w, int32_t ui) const
    {
        Unit::mask_unit(w, ui == 0 ? head : 0, min(Unit::EPU, span - ui * Unit::EPU));
    }
    // unit ui of the row with the neighbours' logits blanked
    __device__ __forceinline__ uint4 load(const uint4 *p, int32_t ui) const
    {
        uint4 w = __ldcs(p + ui);
        if (SHIFTED && touches(ui)) mask(w, ui);
        return w;
    }
};

// One stored logit widened to f32 (T: float, uint16_t = bf16 bits, half_bits = IEEE binary16 bits).
template <typename T>
__device__ __forceinline__ float load_logit(const T *p, size_t i);
template <>
__device__ __forceinline__ float load_logit<float>(const float *p, size_t i) { return __ldcs(p + i); }
template <>
__device__ __forceinline__ float load_logit<uint16_t>(const uint16_t *p, size_t i)
{
    return __uint_as_float(((uint32_t)__ldcs(p + i)) << 16);
}
template <>
__device__ __forceinline__ float load_logit<half_bits>(const half_bits *p, size_t i)
{
    return f16_to_f32(__ldcs(&p[i].bits));
}

// Maximum over the warp in one instruction (sm_100a reduces f32 min/max in hardware).
__device__ __forceinline__ float warp_max(float v)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}

__device__ __forceinline__ double warp_sum_f64(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Reduce a warp's accumulators to one partial (valid in every lane); argmax is left unset.
template <bool REV>
__device__ __forceinline__ RowPartial warp_reduce(RowAcc<REV> acc)
{
    const float Ra = warp_max(acc.rho_a);
    const float Rb = warp_max(acc.rho_b);
    acc.rebase(Ra, Rb);
    RowPartial p;
    p.rho_a = Ra;
    p.rho_b = Rb;
    p.Sa = warp_sum_f64((double)acc.Sa_hi + (double)acc.Sa_lo);
    p.Sb = warp_sum_f64((double)acc.Sb_hi + (double)acc.Sb_lo);
    p.E = warp_sum_f64((double)acc.Et);
    p.D = warp_sum_f64((double)acc.Dt);
    p.B = REV ? warp_sum_f64((double)acc.Bt) : 0.0;
    p.max_a = warp_max(acc.max_a);
    p.argmax = INT32_MAX;
    return p;
}

}  // namespace ppow
