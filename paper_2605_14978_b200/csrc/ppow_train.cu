// Training-side steps next to the scoring pass: group-relative advantage (Sec. 4.1), the sequence form
// of ADAW window scoring with the proportional draw of a window start (Sec. 4.2, Alg. 1), and the expected
// acceptance probability sum_v min(P, Q) (App. B.1).  The first two are tiny; the third streams both
// logit tensors a second time.
#include "../../include/ppow.h"
#include "ppow_device.cuh"
#include "ppow_checked.cuh"

#include <math.h>

namespace ppow {

// ---- group-relative advantage: one warp per rollout group ------------------------------------------
constexpr int ADV_THREADS = 128;

__global__ void __launch_bounds__(ADV_THREADS) group_advantage_kernel(const float *__restrict__ reward, int32_t groups,
                                                                      int32_t G, double delta,
                                                                      float *__restrict__ advantage)
{
    const int lane = threadIdx.x & 31;
    const int32_t g = (int32_t)((blockIdx.x * (unsigned)ADV_THREADS + threadIdx.x) >> 5);
    if (g >= groups) return;
    const float *r = reward + (size_t)g * G;
    double sum = 0.0;
    for (int32_t i = lane; i < G; i += 32) sum += (double)r[i];
    const double mu = warp_sum_f64(sum) / (double)G;
    double sq = 0.0;
    for (int32_t i = lane; i < G; i += 32) {
        const double d = (double)r[i] - mu;
        sq += d * d;
    }
    const double sigma = sqrt(warp_sum_f64(sq) / (double)G);   // population standard deviation
    for (int32_t i = lane; i < G; i += 32)
        advantage[(size_t)g * G + i] = (float)(((double)r[i] - mu) / (sigma + delta));
}

// ---- sequence form of ADAW: one CTA per response ---------------------------------------------------
// Window scores are the plain definition (K additions in index order, float64).  The draw walks the
// running sum of the scores in index order in one thread, chunk by chunk, so that the start it returns
// is decided by exactly the additions the definition names.
constexpr int SEQ_THREADS = 256;

__global__ void __launch_bounds__(SEQ_THREADS) sequence_windows_kernel(const float *__restrict__ crit,
                                                                       const int32_t *__restrict__ seq_offsets,
                                                                       int32_t K, float *__restrict__ scores,
                                                                       const float *__restrict__ uniforms,
                                                                       const float *__restrict__ uniforms_mix,
                                                                       float hard_frac, int32_t *__restrict__ starts)
{
    __shared__ double chunk[SEQ_THREADS];
    __shared__ double total_sh;
    __shared__ int32_t found_sh;

    const int32_t b = (int32_t)blockIdx.x;
    const int32_t o0 = seq_offsets[b], o1 = seq_offsets[b + 1];
    const int32_t T = o1 - o0;
    const int32_t n = T >= K ? T - K + 1 : 0;   // starts with a full window
    const float *v = crit + o0;
    const int tid = threadIdx.x;

    auto score_of = [&](int32_t j) {
        double sum = 0.0;
        if (!PPOW_CHECK(j >= 0 && j + K <= T && o0 >= 0, 401, nullptr)) return 0.0;
        for (int32_t t = j; t < j + K; ++t) sum += (double)v[t];
        return sum / (double)K;
    };

    if (scores) {
        for (int32_t j = tid; j < T; j += SEQ_THREADS) scores[o0 + j] = j < n ? (float)score_of(j) : 0.0f;
    }
    if (!starts) return;
    if (n == 0) {
        if (tid == 0) starts[b] = -1;
        return;
    }
    const double u = (double)uniforms[b];
    // hard-window curriculum: the ADAW draw only when the response's coin falls below hard_frac (strictly),
    // a uniform start otherwise; without a coin array every response takes the ADAW draw
    if (uniforms_mix && !((double)uniforms_mix[b] < (double)hard_frac)) {
        if (tid == 0) {
            const int32_t j = (int32_t)(u * (double)n);
            starts[b] = j < n ? j : n - 1;
        }
        return;
    }

    // pass 1: total of the scores, added in index order
    double run = 0.0;
    for (int32_t c0 = 0; c0 < n; c0 += SEQ_THREADS) {
        const int32_t j = c0 + tid;
        chunk[tid] = j < n ? score_of(j) : 0.0;
        __syncthreads();
        if (tid == 0) {
            const int32_t m = min(SEQ_THREADS, n - c0);
            for (int32_t i = 0; i < m; ++i) run += chunk[i];
        }
        __syncthreads();
    }
    if (tid == 0) {
        total_sh = run;
        found_sh = -1;
    }
    __syncthreads();
    const double total = total_sh;
    if (!(total > 0.0)) {   // no signal anywhere: uniform over the starts
        if (tid == 0) {
            const int32_t j = (int32_t)(u * (double)n);
            starts[b] = j < n ? j : n - 1;
        }
        return;
    }

    // pass 2: first start whose running sum exceeds u * total
    const double thresh = u * total;
    run = 0.0;
    int32_t last_positive = 0;
    for (int32_t c0 = 0; c0 < n; c0 += SEQ_THREADS) {
        const int32_t j = c0 + tid;
        chunk[tid] = j < n ? score_of(j) : 0.0;
        __syncthreads();
        if (tid == 0) {
            const int32_t m = min(SEQ_THREADS, n - c0);
            for (int32_t i = 0; i < m; ++i) {
                run += chunk[i];
                if (chunk[i] > 0.0) last_positive = c0 + i;
                if (run > thresh) {
                    found_sh = c0 + i;
                    break;
                }
            }
        }
        __syncthreads();
        if (found_sh >= 0) break;   // uniform across the block: read after the barrier
    }
    if (tid == 0) starts[b] = found_sh >= 0 ? found_sh : last_positive;   // rounding left the sum at the threshold
}

// ---- expected acceptance: one CTA per (window, position) row ---------------------------------------
constexpr int ACC_THREADS = 256;

// Rows of whole, 16-byte aligned units of any storage format: 16-byte streaming loads, two units of each
// tensor in flight per thread.
template <typename Unit, bool SHIFTED>
__global__ void __launch_bounds__(ACC_THREADS) expected_acceptance_vec_kernel(const uint4 *__restrict__ target,
                                                                              const uint4 *__restrict__ draft,
                                                                              const int32_t *__restrict__ valid_len,
                                                                              const float *__restrict__ lse_p,
                                                                              const float *__restrict__ lse_q, int32_t K,
                                                                              int32_t V, float s,
                                                                              float *__restrict__ out)
{
    __shared__ double warp_part[ACC_THREADS / 32];
    const size_t row = blockIdx.x;
    const int32_t n = (int32_t)(row / (size_t)K), k = (int32_t)(row % (size_t)K);
    const int tid = threadIdx.x;
    if (valid_len && k >= valid_len[n]) {
        if (tid == 0) out[row] = 0.0f;
        return;
    }
    // P(v) = 2^(a*s - la), Q(v) = 2^(b*s - lb) with the normalisers converted to log2 units
    const float la = lse_p[row] * 1.4426950408889634f, lb = lse_q[row] * 1.4426950408889634f;
    // rows may start inside a 16-byte unit (odd V, offset base): both tensors at the same offset; the logits of
    // the first and last unit that belong to the neighbouring rows are blanked (they then add min(0, 0))
    const RowSpan<Unit, SHIFTED> ra(target, row, V), rb(draft, row, V);
    const uint4 *pa = ra.base, *pb = rb.base;
    const int32_t units = ra.units;
    float acc0 = 0.0f, acc1 = 0.0f;
    if (!PPOW_CHECK(row < (size_t)gridDim.x && k < K && ra.head == rb.head, 402, nullptr)) return;
    auto add_unit = [&](const uint4 &A, const uint4 &B) {
        float fa[Unit::EPU], fb[Unit::EPU];
        Unit::unpack(A, fa);
        Unit::unpack(B, fb);
#pragma unroll
        for (int e = 0; e < Unit::EPU; e += 2) {
            acc0 += fminf(ex2_approx(fmaf(fa[e], s, -la)), ex2_approx(fmaf(fb[e], s, -lb)));
            acc1 += fminf(ex2_approx(fmaf(fa[e + 1], s, -la)), ex2_approx(fmaf(fb[e + 1], s, -lb)));
        }
    };
    int32_t u = tid;
    for (; u + ACC_THREADS < units; u += 2 * ACC_THREADS) {
        const uint4 A0 = ra.load(pa, u), B0 = rb.load(pb, u);
        const uint4 A1 = ra.load(pa, u + ACC_THREADS), B1 = rb.load(pb, u + ACC_THREADS);
        add_unit(A0, B0);
        add_unit(A1, B1);
    }
    if (u < units) add_unit(ra.load(pa, u), rb.load(pb, u));
    const double w = warp_sum_f64((double)acc0 + (double)acc1);
    if ((tid & 31) == 0) warp_part[tid >> 5] = w;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
#pragma unroll
        for (int i = 0; i < ACC_THREADS / 32; ++i) t += warp_part[i];
        out[row] = (float)fmin(t, 1.0);
    }
}

// Any V, any alignment: one logit per load.
template <typename T>
__global__ void __launch_bounds__(ACC_THREADS) expected_acceptance_scalar_kernel(const T *__restrict__ target,
                                                                                 const T *__restrict__ draft,
                                                                                 const int32_t *__restrict__ valid_len,
                                                                                 const float *__restrict__ lse_p,
                                                                                 const float *__restrict__ lse_q, int32_t K,
                                                                                 int32_t V, float s, float *__restrict__ out)
{
    __shared__ double warp_part[ACC_THREADS / 32];
    const size_t row = blockIdx.x;
    const int32_t n = (int32_t)(row / (size_t)K), k = (int32_t)(row % (size_t)K);
    const int tid = threadIdx.x;
    if (valid_len && k >= valid_len[n]) {
        if (tid == 0) out[row] = 0.0f;
        return;
    }
    const float la = lse_p[row] * 1.4426950408889634f, lb = lse_q[row] * 1.4426950408889634f;
    const T *pa = target + row * (size_t)V, *pb = draft + row * (size_t)V;
    float acc = 0.0f;
    for (int32_t v = tid; v < V; v += ACC_THREADS)
        acc += fminf(ex2_approx(fmaf(load_logit<T>(pa, v), s, -la)), ex2_approx(fmaf(load_logit<T>(pb, v), s, -lb)));
    const double w = warp_sum_f64((double)acc);
    if ((tid & 31) == 0) warp_part[tid >> 5] = w;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
#pragma unroll
        for (int i = 0; i < ACC_THREADS / 32; ++i) t += warp_part[i];
        out[row] = (float)fmin(t, 1.0);
    }
}

// ---- log-probability of the reference window ---------------------------------------------------------
// Per row: log2-domain sum of 2^(v*s - rho) against a stale per-thread reference (raised only when a
// group of logits exceeds it by 2^4), group-local f32 partial folded into a compensated (hi, lo) pair,
// merged across the block in float64.  log max_v P(v) = ln2 * (M*s - R - log2 S).
constexpr int REF_THREADS = 256;

struct LseAcc {
    float rho, S, S_hi, S_lo, m;

    __device__ __forceinline__ void reset()
    {
        rho = -1.0e30f;
        S = S_hi = S_lo = 0.0f;
        m = -INFINITY;
    }
    __device__ __forceinline__ void fold()
    {
        const float t = S_hi + S, bp = t - S_hi;
        S_lo += (S_hi - (t - bp)) + (S - bp);
        S_hi = t;
        S = 0.0f;
    }
    __device__ __forceinline__ void guard(float group_max, float s)
    {
        m = fmaxf(m, group_max);
        if (fmaf(group_max, s, -rho) > 4.0f) {
            fold();
            const float nr = group_max * s, f = ex2_approx(rho - nr);
            S_hi *= f;
            S_lo *= f;
            rho = nr;
        }
    }
    __device__ __forceinline__ void add(float v, float s) { S += ex2_approx(fmaf(v, s, -rho)); }
};

// Block merge of the per-thread sums against the largest reference; thread 0 writes the row's value.
__device__ __forceinline__ void lse_block_finish(const LseAcc &acc, float s, float *row_logp_out)
{
    __shared__ float sh_rho[REF_THREADS / 32], sh_m[REF_THREADS / 32];
    __shared__ double sh_S[REF_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float R = warp_max(acc.rho), M = warp_max(acc.m);
    const double Sw = warp_sum_f64(exp2((double)acc.rho - (double)R) * ((double)acc.S_hi + (double)acc.S_lo));
    if (lane == 0) {
        sh_rho[warp] = R;
        sh_m[warp] = M;
        sh_S[warp] = Sw;
    }
    __syncthreads();
    if (tid == 0) {
        float Rb = sh_rho[0], Mb = sh_m[0];
#pragma unroll
        for (int i = 1; i < REF_THREADS / 32; ++i) {
            Rb = fmaxf(Rb, sh_rho[i]);
            Mb = fmaxf(Mb, sh_m[i]);
        }
        double Sb = 0.0;
#pragma unroll
        for (int i = 0; i < REF_THREADS / 32; ++i) Sb += exp2((double)sh_rho[i] - (double)Rb) * sh_S[i];
        *row_logp_out = (float)((fma((double)Mb, (double)s, -(double)Rb) - log2(Sb)) * 0.69314718055994530942);
    }
}

// One CTA per (window, position) row from a plain grid; writes log max_v P(v) of the row.
// Rows of whole, 16-byte aligned units of any storage format (one fold per 8 or 16 logits).
template <typename Unit, bool SHIFTED>
__global__ void __launch_bounds__(REF_THREADS) reference_logprob_vec_kernel(const uint4 *__restrict__ ref,
                                                                            const int32_t *__restrict__ valid_len,
                                                                            int32_t K, int32_t V, float s,
                                                                            float *__restrict__ row_logp)
{
    const size_t row = blockIdx.x;
    const int32_t n = (int32_t)(row / (size_t)K), k = (int32_t)(row % (size_t)K);
    const int tid = threadIdx.x;
    if (valid_len && k >= valid_len[n]) {
        if (tid == 0) row_logp[row] = 0.0f;
        return;
    }
    LseAcc acc;
    acc.reset();
    const RowSpan<Unit, SHIFTED> rs(ref, row, V);   // the row may start inside a 16-byte unit: first and last unit are blanked
    const uint4 *p = rs.base;
    const int32_t units = rs.units;
    auto add_unit = [&](const uint4 &w) {
        float f[Unit::EPU];
        Unit::unpack(w, f);
#pragma unroll
        for (int e = 0; e < Unit::EPU; ++e) acc.add(f[e], s);
    };
    // four units of the row in flight per thread (a single tensor is read: fewer loads per thread would leave
    // the memory system short of requests), one reference check and one fold per round
    int32_t u = tid;
    for (; u + 3 * REF_THREADS < units; u += 4 * REF_THREADS) {
        const uint4 w0 = rs.load(p, u), w1 = rs.load(p, u + REF_THREADS);
        const uint4 w2 = rs.load(p, u + 2 * REF_THREADS), w3 = rs.load(p, u + 3 * REF_THREADS);
        acc.guard(fmaxf(fmaxf(Unit::unit_max(w0), Unit::unit_max(w1)), fmaxf(Unit::unit_max(w2), Unit::unit_max(w3))), s);
        add_unit(w0);
        add_unit(w1);
        acc.fold();
        add_unit(w2);
        add_unit(w3);
        acc.fold();
    }
    for (; u < units; u += REF_THREADS) {
        const uint4 w0 = rs.load(p, u);
        acc.guard(Unit::unit_max(w0), s);
        add_unit(w0);
        acc.fold();
    }
    lse_block_finish(acc, s, row_logp + row);
}

// ref_logp[n] = sum of the window's row values, added in position order (float64).
__global__ void reference_logprob_sum_kernel(const float *__restrict__ row_logp, const int32_t *__restrict__ valid_len,
                                             int32_t N, int32_t K, float *__restrict__ ref_logp)
{
    const int32_t n = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x);
    if (n >= N) return;
    int32_t L = valid_len ? valid_len[n] : K;
    L = max(0, min(L, K));
    double sum = 0.0;
    for (int32_t t = 0; t < L; ++t) sum += (double)row_logp[(size_t)n * K + t];
    ref_logp[n] = (float)sum;
}

}  // namespace ppow

using namespace ppow;

#ifdef PPOW_CHECKED
namespace ppow { int read_check_counters_train(unsigned int *f, unsigned int *s) { return read_check_counters(f, s); } }
#endif

extern "C" ppow_status ppow_group_advantage(const float *reward, int32_t N, int32_t group_size, float delta,
                                            float *advantage, void *cuda_stream)
{
    if (N < 0 || group_size < 1 || group_size > 1024 || N % group_size != 0) return PPOW_ERR_INVALID_ARG;
    if (!(delta >= 0.0f) || !isfinite(delta)) return PPOW_ERR_INVALID_ARG;
    if (N == 0) return PPOW_OK;
    if (!reward || !advantage || reward == advantage) return PPOW_ERR_INVALID_ARG;
    const int32_t groups = N / group_size;
    const unsigned grid = (unsigned)(((size_t)groups * 32 + ADV_THREADS - 1) / ADV_THREADS);
    group_advantage_kernel<<<grid, ADV_THREADS, 0, (cudaStream_t)cuda_stream>>>(reward, groups, group_size, (double)delta,
                                                                               advantage);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

extern "C" ppow_status ppow_sequence_windows(const float *crit, const int32_t *seq_offsets, int32_t B, int32_t K,
                                             float *scores, const float *uniforms, int32_t *starts, void *cuda_stream)
{
    if (B < 0 || K < 1 || K > 1024) return PPOW_ERR_INVALID_ARG;
    if (B == 0) return PPOW_OK;
    if (!crit || !seq_offsets) return PPOW_ERR_INVALID_ARG;
    if (starts && !uniforms) return PPOW_ERR_INVALID_ARG;
    if (!scores && !starts) return PPOW_OK;
    sequence_windows_kernel<<<(unsigned)B, SEQ_THREADS, 0, (cudaStream_t)cuda_stream>>>(crit, seq_offsets, K, scores,
                                                                                      uniforms, nullptr, 1.0f, starts);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

extern "C" ppow_status ppow_sequence_windows_mixed(const float *crit, const int32_t *seq_offsets, int32_t B, int32_t K,
                                                   float hard_frac, float *scores, const float *uniforms_mix,
                                                   const float *uniforms_draw, int32_t *starts, void *cuda_stream)
{
    if (B < 0 || K < 1 || K > 1024) return PPOW_ERR_INVALID_ARG;
    if (!(hard_frac >= 0.0f) || !(hard_frac <= 1.0f)) return PPOW_ERR_INVALID_ARG;
    if (B == 0) return PPOW_OK;
    if (!crit || !seq_offsets) return PPOW_ERR_INVALID_ARG;
    if (starts && (!uniforms_mix || !uniforms_draw)) return PPOW_ERR_INVALID_ARG;
    if (!scores && !starts) return PPOW_OK;
    sequence_windows_kernel<<<(unsigned)B, SEQ_THREADS, 0, (cudaStream_t)cuda_stream>>>(
        crit, seq_offsets, K, scores, uniforms_draw, uniforms_mix, hard_frac, starts);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

extern "C" ppow_status ppow_expected_acceptance(const ppow_params *params,
                                                const void *draft_logits, const void *target_logits,
                                                const int32_t *valid_len, const float *lse_p, const float *lse_q,
                                                float *expected_accept, void *cuda_stream)
{
    if (!params || params->N < 0 || params->K < 1 || params->V < 2) return PPOW_ERR_INVALID_ARG;
    if (params->dtype != PPOW_F32 && params->dtype != PPOW_BF16 && params->dtype != PPOW_F16) return PPOW_ERR_INVALID_ARG;
    if (!(params->temperature > 0.0f) || !isfinite(params->temperature)) return PPOW_ERR_INVALID_ARG;
    if ((int64_t)params->N * params->K > (int64_t)1 << 26) return PPOW_ERR_INVALID_ARG;
    if (params->N == 0) return PPOW_OK;
    if (!draft_logits || !target_logits || !lse_p || !lse_q || !expected_accept) return PPOW_ERR_INVALID_ARG;
    const size_t esize = params->dtype == PPOW_F32 ? 4 : 2;
    if (((uintptr_t)draft_logits % esize) || ((uintptr_t)target_logits % esize)) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const unsigned rows = (unsigned)((size_t)params->N * params->K);
    const float s = (float)(1.4426950408889634074 / (double)params->temperature);
    const int32_t K = params->K, V = params->V;
    const int epu = params->dtype == PPOW_F32 ? 4 : 8;
    const bool vec = (uintptr_t)draft_logits % 16 == (uintptr_t)target_logits % 16;   // same offset within a 16-byte unit
    const uint4 *ta = (const uint4 *)target_logits, *da = (const uint4 *)draft_logits;
    const bool shifted = V % epu != 0 || (uintptr_t)target_logits % 16 != 0;   // rows that start inside a unit
#define PPOW_ACC(UNIT)                                                                                          \
    do {                                                                                                        \
        if (shifted)                                                                                            \
            expected_acceptance_vec_kernel<UNIT, true><<<rows, ACC_THREADS, 0, stream>>>(ta, da, valid_len, lse_p, lse_q, K, \
                                                                                          V, s, expected_accept); \
        else                                                                                                    \
            expected_acceptance_vec_kernel<UNIT, false><<<rows, ACC_THREADS, 0, stream>>>(ta, da, valid_len, lse_p, lse_q, K, \
                                                                                           V, s, expected_accept); \
    } while (0)
    if (vec && params->dtype == PPOW_BF16)
        PPOW_ACC(UnitBf16);
    else if (vec && params->dtype == PPOW_F16)
        PPOW_ACC(UnitF16);
    else if (vec)
        PPOW_ACC(UnitF32);
#undef PPOW_ACC
    else if (params->dtype == PPOW_F32)
        expected_acceptance_scalar_kernel<float><<<rows, ACC_THREADS, 0, stream>>>(
            (const float *)target_logits, (const float *)draft_logits, valid_len, lse_p, lse_q, K, V, s, expected_accept);
    else if (params->dtype == PPOW_F16)
        expected_acceptance_scalar_kernel<half_bits><<<rows, ACC_THREADS, 0, stream>>>(
            (const half_bits *)target_logits, (const half_bits *)draft_logits, valid_len, lse_p, lse_q, K, V, s, expected_accept);
    else
        expected_acceptance_scalar_kernel<uint16_t><<<rows, ACC_THREADS, 0, stream>>>(
            (const uint16_t *)target_logits, (const uint16_t *)draft_logits, valid_len, lse_p, lse_q, K, V, s, expected_accept);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

extern "C" ppow_status ppow_reference_logprob(const ppow_params *params, const void *ref_target_logits,
                                              const int32_t *valid_len, float *row_logp, float *ref_logp,
                                              void *cuda_stream)
{
    if (!params || params->N < 0 || params->K < 1 || params->V < 2) return PPOW_ERR_INVALID_ARG;
    if (params->dtype != PPOW_F32 && params->dtype != PPOW_BF16 && params->dtype != PPOW_F16) return PPOW_ERR_INVALID_ARG;
    if (!(params->temperature > 0.0f) || !isfinite(params->temperature)) return PPOW_ERR_INVALID_ARG;
    if ((int64_t)params->N * params->K > (int64_t)1 << 26) return PPOW_ERR_INVALID_ARG;
    if (params->N == 0) return PPOW_OK;
    if (!ref_target_logits || !row_logp) return PPOW_ERR_INVALID_ARG;
    const size_t esize = params->dtype == PPOW_F32 ? 4 : 2;
    if ((uintptr_t)ref_target_logits % esize) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const float s = (float)(1.4426950408889634074 / (double)params->temperature);
    const unsigned rows = (unsigned)((size_t)params->N * params->K);
    const int32_t K = params->K, V = params->V;
    // any V and any element-aligned base: rows that start inside a 16-byte unit are masked at their ends
    const uint4 *ra = (const uint4 *)ref_target_logits;
    const bool shifted = V % (params->dtype == PPOW_F32 ? 4 : 8) != 0 || (uintptr_t)ref_target_logits % 16 != 0;
#define PPOW_REF(UNIT)                                                                                                   \
    do {                                                                                                                 \
        if (shifted)                                                                                                     \
            reference_logprob_vec_kernel<UNIT, true><<<rows, REF_THREADS, 0, stream>>>(ra, valid_len, K, V, s, row_logp); \
        else                                                                                                             \
            reference_logprob_vec_kernel<UNIT, false><<<rows, REF_THREADS, 0, stream>>>(ra, valid_len, K, V, s, row_logp); \
    } while (0)
    if (params->dtype == PPOW_BF16)
        PPOW_REF(UnitBf16);
    else if (params->dtype == PPOW_F16)
        PPOW_REF(UnitF16);
    else
        PPOW_REF(UnitF32);
#undef PPOW_REF
    if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
    if (ref_logp) {
        reference_logprob_sum_kernel<<<(unsigned)((params->N + 127) / 128), 128, 0, stream>>>(row_logp, valid_len, params->N,
                                                                                             params->K, ref_logp);
        if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
    }
    return PPOW_OK;
}
