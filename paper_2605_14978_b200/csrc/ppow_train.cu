// Training-side steps next to the scoring pass: group-relative advantage (Sec. 4.1), the sequence form
// of ADAW window scoring with the proportional draw of a window start (Sec. 4.2, Alg. 1), and the expected
// acceptance probability sum_v min(P, Q) (App. B.1).  The first two are tiny; the third streams both
// logit tensors a second time.
#include "../../include/ppow.h"

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace ppow {

__device__ __forceinline__ double warp_sum_double(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

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
    const double mu = warp_sum_double(sum) / (double)G;
    double sq = 0.0;
    for (int32_t i = lane; i < G; i += 32) {
        const double d = (double)r[i] - mu;
        sq += d * d;
    }
    const double sigma = sqrt(warp_sum_double(sq) / (double)G);   // population standard deviation
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

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T>
__device__ __forceinline__ float logit_at(const T *p, size_t i);
template <>
__device__ __forceinline__ float logit_at<float>(const float *p, size_t i) { return __ldcs(p + i); }
template <>
__device__ __forceinline__ float logit_at<uint16_t>(const uint16_t *p, size_t i)   // bf16 bit patterns
{
    return __uint_as_float(((uint32_t)__ldcs(p + i)) << 16);
}
struct half_bits {   // IEEE binary16 bit patterns
    uint16_t bits;
};
template <>
__device__ __forceinline__ float logit_at<half_bits>(const half_bits *p, size_t i)
{
    return __half2float(__ushort_as_half(__ldcs(&p[i].bits)));
}

// VEC: bf16 rows of whole, 16-byte aligned 8-logit units.
template <typename T, bool VEC>
__global__ void __launch_bounds__(ACC_THREADS) expected_acceptance_kernel(const T *__restrict__ target,
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
    // P(v) = 2^(a*s - la), Q(v) = 2^(b*s - lb) with the normalisers converted to log2 units
    const float la = lse_p[row] * 1.4426950408889634f, lb = lse_q[row] * 1.4426950408889634f;
    float acc0 = 0.0f, acc1 = 0.0f;
    if (VEC) {
        const uint4 *pa = reinterpret_cast<const uint4 *>(target) + row * (size_t)(V >> 3);
        const uint4 *pb = reinterpret_cast<const uint4 *>(draft) + row * (size_t)(V >> 3);
        for (int32_t u = tid; u < (V >> 3); u += ACC_THREADS) {
            const uint4 A = __ldcs(pa + u), B = __ldcs(pb + u);
            const uint32_t wa[4] = {A.x, A.y, A.z, A.w}, wb[4] = {B.x, B.y, B.z, B.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float p0 = ex2f(fmaf(__uint_as_float(wa[q] << 16), s, -la));
                const float q0 = ex2f(fmaf(__uint_as_float(wb[q] << 16), s, -lb));
                const float p1 = ex2f(fmaf(__uint_as_float(wa[q] & 0xffff0000u), s, -la));
                const float q1 = ex2f(fmaf(__uint_as_float(wb[q] & 0xffff0000u), s, -lb));
                acc0 += fminf(p0, q0);
                acc1 += fminf(p1, q1);
            }
        }
    } else {
        const T *pa = target + row * (size_t)V, *pb = draft + row * (size_t)V;
        for (int32_t v = tid; v < V; v += ACC_THREADS)
            acc0 += fminf(ex2f(fmaf(logit_at<T>(pa, v), s, -la)), ex2f(fmaf(logit_at<T>(pb, v), s, -lb)));
    }
    const double w = warp_sum_double((double)acc0 + (double)acc1);
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

__device__ __forceinline__ uint32_t max_bf16x2_(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

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
            const float nr = group_max * s, f = ex2f(rho - nr);
            S_hi *= f;
            S_lo *= f;
            rho = nr;
        }
    }
    __device__ __forceinline__ void add(float v, float s) { S += ex2f(fmaf(v, s, -rho)); }
};

// One CTA per (window, position) row from a plain grid; writes log max_v P(v) of the row.
template <typename T, bool VEC>
__global__ void __launch_bounds__(REF_THREADS) reference_logprob_rows_kernel(const T *__restrict__ ref,
                                                                             const int32_t *__restrict__ valid_len,
                                                                             int32_t K, int32_t V, float s,
                                                                             float *__restrict__ row_logp)
{
    __shared__ float sh_rho[REF_THREADS / 32], sh_m[REF_THREADS / 32];
    __shared__ double sh_S[REF_THREADS / 32];
    const size_t row = blockIdx.x;
    const int32_t n = (int32_t)(row / (size_t)K), k = (int32_t)(row % (size_t)K);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (valid_len && k >= valid_len[n]) {
        if (tid == 0) row_logp[row] = 0.0f;
        return;
    }
    LseAcc acc;
    acc.reset();
    if (VEC) {
        const uint4 *p = reinterpret_cast<const uint4 *>(ref) + row * (size_t)(V >> 3);
        const int32_t units = V >> 3;
        for (int32_t u = tid; u < units; u += 2 * REF_THREADS) {
            const bool two = u + REF_THREADS < units;
            const uint4 w0 = __ldcs(p + u);
            const uint4 w1 = two ? __ldcs(p + u + REF_THREADS) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
            uint32_t mx = max_bf16x2_(max_bf16x2_(max_bf16x2_(w0.x, w0.y), max_bf16x2_(w0.z, w0.w)),
                                      max_bf16x2_(max_bf16x2_(w1.x, w1.y), max_bf16x2_(w1.z, w1.w)));
            acc.guard(fmaxf(__uint_as_float(mx << 16), __uint_as_float(mx & 0xffff0000u)), s);
            const uint32_t w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (q < 4 || two) {
                    acc.add(__uint_as_float(w[q] << 16), s);
                    acc.add(__uint_as_float(w[q] & 0xffff0000u), s);
                }
            }
            acc.fold();
        }
    } else {
        const T *p = ref + row * (size_t)V;
        for (int32_t i = tid; i < V; i += REF_THREADS) {
            const float v = logit_at<T>(p, i);
            acc.guard(v, s);
            acc.add(v, s);
            acc.fold();
        }
    }
    // block merge against the largest reference
    float R = acc.rho, M = acc.m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        R = fmaxf(R, __shfl_xor_sync(0xffffffffu, R, o));
        M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    }
    const double Sw = warp_sum_double(exp2((double)acc.rho - (double)R) * ((double)acc.S_hi + (double)acc.S_lo));
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
        row_logp[row] = (float)((fma((double)Mb, (double)s, -(double)Rb) - log2(Sb)) * 0.69314718055994530942);
    }
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
    if (params->dtype == PPOW_F32) {
        expected_acceptance_kernel<float, false><<<rows, ACC_THREADS, 0, stream>>>(
            (const float *)target_logits, (const float *)draft_logits, valid_len, lse_p, lse_q, K, V, s, expected_accept);
    } else if (params->dtype == PPOW_F16) {
        expected_acceptance_kernel<half_bits, false><<<rows, ACC_THREADS, 0, stream>>>(
            (const half_bits *)target_logits, (const half_bits *)draft_logits, valid_len, lse_p, lse_q, K, V, s,
            expected_accept);
    } else if (V % 8 == 0 && (uintptr_t)draft_logits % 16 == 0 && (uintptr_t)target_logits % 16 == 0) {
        expected_acceptance_kernel<uint16_t, true><<<rows, ACC_THREADS, 0, stream>>>(
            (const uint16_t *)target_logits, (const uint16_t *)draft_logits, valid_len, lse_p, lse_q, K, V, s,
            expected_accept);
    } else {
        expected_acceptance_kernel<uint16_t, false><<<rows, ACC_THREADS, 0, stream>>>(
            (const uint16_t *)target_logits, (const uint16_t *)draft_logits, valid_len, lse_p, lse_q, K, V, s,
            expected_accept);
    }
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
    if (params->dtype == PPOW_F32)
        reference_logprob_rows_kernel<float, false><<<rows, REF_THREADS, 0, stream>>>(
            (const float *)ref_target_logits, valid_len, params->K, params->V, s, row_logp);
    else if (params->dtype == PPOW_F16)
        reference_logprob_rows_kernel<half_bits, false><<<rows, REF_THREADS, 0, stream>>>(
            (const half_bits *)ref_target_logits, valid_len, params->K, params->V, s, row_logp);
    else if (params->V % 8 == 0 && (uintptr_t)ref_target_logits % 16 == 0)
        reference_logprob_rows_kernel<uint16_t, true><<<rows, REF_THREADS, 0, stream>>>(
            (const uint16_t *)ref_target_logits, valid_len, params->K, params->V, s, row_logp);
    else
        reference_logprob_rows_kernel<uint16_t, false><<<rows, REF_THREADS, 0, stream>>>(
            (const uint16_t *)ref_target_logits, valid_len, params->K, params->V, s, row_logp);
    if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
    if (ref_logp) {
        reference_logprob_sum_kernel<<<(unsigned)((params->N + 127) / 128), 128, 0, stream>>>(row_logp, valid_len, params->N,
                                                                                             params->K, ref_logp);
        if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
    }
    return PPOW_OK;
}
