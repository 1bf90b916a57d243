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
// Accumulating D from the per-element difference (not E - F) avoids cancelling two O(10) terms
// to reach a KL of O(0.01).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ppow {

constexpr float REBASE_LOG2 = 4.0f;      // raise a reference when a tile exceeds it by 2^4
constexpr float RHO_INIT = -1.0e30f;     // "no reference yet": the first tile always rebases

// One partial reduction of (part of) a row; merged later in float64.
struct __align__(16) RowPartial {
    float rho_a, rho_b;   // references, log2 units
    float Sa, Sb;         // sums relative to those references (leading parts)
    float Sa_lo, Sb_lo;   // their compensation terms: the sums are Sa + Sa_lo, Sb + Sb_lo
    float E, D;
    float max_a;          // largest stored target logit seen
    int32_t argmax;       // its lowest vocabulary index
    int32_t pad[2];
};
static_assert(sizeof(RowPartial) == 48, "RowPartial layout");

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
// Sa and Sb are what log-probabilities are read from, and a confident distribution puts almost all
// of a sum into one term: once an f32 accumulator holds that term, every later small term is rounded
// at its ulp (6e-8 relative each, hundreds of times).  So both sums are kept as tile-local partials
// (Sa[], Sb[], restarted from zero by flush()) that are folded into a running (hi, lo) pair with an
// error-compensated add; only the few adds inside one tile can be absorbed.
struct RowAcc {
    float rho_a, rho_b;
    float Sa[2], Sb[2], E[2], D[2];
    float Sa_hi, Sa_lo, Sb_hi, Sb_lo;
    float max_a;
    int32_t best;       // where max_a was first seen (meaning defined by the caller)

    __device__ __forceinline__ void reset()
    {
        rho_a = rho_b = RHO_INIT;
        Sa[0] = Sa[1] = Sb[0] = Sb[1] = E[0] = E[1] = D[0] = D[1] = 0.0f;
        Sa_hi = Sa_lo = Sb_hi = Sb_lo = 0.0f;
        max_a = -INFINITY;
        best = 0;
    }

    // Fold the tile-local partial sums into the compensated running sums (call once per tile).
    __device__ __forceinline__ void flush()
    {
        const float pa = Sa[0] + Sa[1], pb = Sb[0] + Sb[1];
        const float ta = Sa_hi + pa, tb = Sb_hi + pb;
        Sa_lo += pa - (ta - Sa_hi);
        Sb_lo += pb - (tb - Sb_hi);
        Sa_hi = ta;
        Sb_hi = tb;
        Sa[0] = Sa[1] = Sb[0] = Sb[1] = 0.0f;
    }

    // Move both references (log2 units).  Only between tiles (after flush()).  With x' = x - d,
    //   Sa' = fa*Sa,  E' = fa*(E + da*Sa),  D' = fa*(D + (da - db)*Sa),  Sb' = fb*Sb
    // where da = rho_a - new_rho_a <= 0 and fa = 2^da (same for b).  Applying (da - db) in one step
    // keeps D exactly 0 when draft and target are the same data.
    __device__ __forceinline__ void rebase(float new_rho_a, float new_rho_b)
    {
        const float da = rho_a - new_rho_a, db = rho_b - new_rho_b;
        const float fa = ex2_approx(da), fb = ex2_approx(db);
        const float S = Sa_hi + Sa_lo;
        E[0] = fa * fmaf(da, S, E[0] + E[1]);
        D[0] = fa * fmaf(da - db, S, D[0] + D[1]);
        E[1] = D[1] = 0.0f;
        Sa_hi *= fa;
        Sa_lo *= fa;
        Sb_hi *= fb;
        Sb_lo *= fb;
        rho_a = new_rho_a;
        rho_b = new_rho_b;
    }

    // One (target, draft) pair already widened to f32.  i selects the accumulator set.
    __device__ __forceinline__ void add_pair(float a, float b, float s, int i)
    {
        const float xa = fmaf(a, s, -rho_a);
        const float xb = fmaf(b, s, -rho_b);
        const float ea = ex2_approx(xa);
        const float eb = ex2_approx(xb);
        Sa[i] += ea;
        Sb[i] += eb;
        E[i] = fmaf(ea, xa, E[i]);
        D[i] = fmaf(ea, xa - xb, D[i]);
    }

    // Two packed bf16 pairs.
    __device__ __forceinline__ void add_word(uint32_t wa, uint32_t wb, float s)
    {
        add_pair(bf16_lo(wa), bf16_lo(wb), s, 0);
        add_pair(bf16_hi(wa), bf16_hi(wb), s, 1);
    }

    // Raise the references if this tile's maxima (raw logit units) call for it.
    __device__ __forceinline__ void guard(float tile_max_a, float tile_max_b, float s)
    {
        const bool up_a = fmaf(tile_max_a, s, -rho_a) > REBASE_LOG2;
        const bool up_b = fmaf(tile_max_b, s, -rho_b) > REBASE_LOG2;
        if (up_a | up_b) rebase(up_a ? tile_max_a * s : rho_a, up_b ? tile_max_b * s : rho_b);
    }

    __device__ __forceinline__ void fold()
    {
        E[0] += E[1]; D[0] += D[1];
        E[1] = D[1] = 0.0f;
    }
};

// Error-compensated sum of (hi, lo) pairs across a warp; every lane ends with the same pair.
__device__ __forceinline__ void warp_sum_pair(float &hi, float &lo)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float oh = __shfl_xor_sync(0xffffffffu, hi, o);
        const float ol = __shfl_xor_sync(0xffffffffu, lo, o);
        const float big = fmaxf(hi, oh), small = fminf(hi, oh);   // sums of 2^x are non-negative
        const float t = big + small;
        lo = (lo + ol) + (small - (t - big));
        hi = t;
    }
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Reduce a warp's accumulators to one partial (valid in every lane); argmax is left unset.
__device__ __forceinline__ RowPartial warp_reduce(RowAcc acc)
{
    acc.fold();
    const float Ra = warp_max(acc.rho_a);
    const float Rb = warp_max(acc.rho_b);
    acc.rebase(Ra, Rb);
    RowPartial p;
    p.rho_a = Ra;
    p.rho_b = Rb;
    warp_sum_pair(acc.Sa_hi, acc.Sa_lo);
    warp_sum_pair(acc.Sb_hi, acc.Sb_lo);
    p.Sa = acc.Sa_hi; p.Sa_lo = acc.Sa_lo;
    p.Sb = acc.Sb_hi; p.Sb_lo = acc.Sb_lo;
    p.pad[0] = p.pad[1] = 0;
    p.E = warp_sum(acc.E[0]);
    p.D = warp_sum(acc.D[0]);
    p.max_a = warp_max(acc.max_a);
    p.argmax = INT32_MAX;
    return p;
}

__device__ __forceinline__ RowAcc acc_from_partial(const RowPartial &p)
{
    RowAcc a;
    a.reset();
    a.rho_a = p.rho_a; a.rho_b = p.rho_b;
    a.Sa_hi = p.Sa; a.Sa_lo = p.Sa_lo; a.Sb_hi = p.Sb; a.Sb_lo = p.Sb_lo; a.E[0] = p.E; a.D[0] = p.D;
    a.max_a = p.max_a;
    return a;
}

}  // namespace ppow
