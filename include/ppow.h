/*
 * ppow.h -- C ABI of the B200 (sm_100a) PPOW window-scoring library.
 *
 * Scores N speculative windows of K drafted positions over a vocabulary of V entries from paired
 * draft and target logits, then ranks windows for Adaptive Divergence-Aware Windowing.
 *
 * Conventions that hold for every entry point unless it says otherwise
 *   - "device" pointers address memory of the CUDA device that is current when the call is made;
 *     "host" pointers address ordinary host memory.  The library never takes ownership of a buffer.
 *   - The library allocates no device memory.  Scratch space is passed in as `workspace`
 *     (query its size with the matching *_workspace_bytes function; 256-byte alignment required).
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t, NULL = the legacy default stream)
 *     and return without synchronising.  Inputs are read-only.  Calls on different streams must
 *     use different workspaces.
 *   - Host-detectable problems return an error status before anything is launched; nothing is
 *     printed and the process is never aborted.
 *   - Logits must be finite.  Layout of logits is [N, K, V] row-major with the vocabulary
 *     contiguous; per-position arrays are [N, K] row-major; per-window arrays are [N].
 */
#ifndef PPOW_H_
#define PPOW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PPOW_OK = 0,
    PPOW_ERR_INVALID_ARG = 1,   /* null/misaligned pointer, size or parameter out of range */
    PPOW_ERR_UNSUPPORTED = 2,   /* valid request the library cannot serve (e.g. K > 32) */
    PPOW_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small */
    PPOW_ERR_CUDA = 4,          /* a CUDA runtime call or kernel launch failed */
    PPOW_ERR_DEVICE_TIMEOUT = 5 /* a bounded device-side wait gave up (reported by ppow_read_error_flags) */
} ppow_status;

/* Acceptance test.  PPOW_STOCHASTIC is rejection-sampling verification: accept position t iff
 * u_t <= min(1, P_t(yhat_t)/Q_t(yhat_t)) (App. C.1).  PPOW_GREEDY is its temperature-0 decoding
 * case: accept iff yhat_t is the target's most likely token (Sec. 5.1, decoding temperatures 0 and 1;
 * Fig. 1).  The mode changes only the acceptance test; entropy, KL and Delta always use
 * `temperature`. */
typedef enum { PPOW_GREEDY = 0, PPOW_STOCHASTIC = 1 } ppow_mode;

typedef enum { PPOW_F32 = 0, PPOW_BF16 = 1, PPOW_F16 = 2 } ppow_dtype;   /* storage type of the logits */

/* Bits of the device-side error word (ppow_read_error_flags). */
enum {
    PPOW_FLAG_TOKEN_RANGE = 1u,   /* some draft token was outside [0, V): that position was rejected */
    PPOW_FLAG_DEVICE_TIMEOUT = 2u, /* a bounded wait inside a kernel ran out */
    PPOW_FLAG_BOUNDS = 4u          /* bounds-checked build only: an index computed by a kernel was out of range
                                      (the access was skipped; see ppow_checked_failures) */
};

typedef struct {
    int32_t N;           /* windows, >= 0 */
    int32_t K;           /* drafted positions per window, 1..32 (the paper trains with K = 10) */
    int32_t V;           /* vocabulary size, >= 2 */
    int32_t dtype;       /* ppow_dtype of both logit tensors */
    int32_t mode;        /* ppow_mode */
    float c;             /* relative drafter cost gamma >= 0 in R_speedup = k/(k*gamma + 1) (Sec. 4.3.1) */
    float temperature;   /* T > 0; P_t = softmax(target/T), Q_t = softmax(draft/T) (Sec. 4.2) */
    float eta;           /* scale of the Distribution-Based Proximity Reward (Sec. 4.3.2; paper: 1.0) */
    float eps;           /* its tolerance: R_dist = eta * 1[k = 0] * 1[Delta < eps] (paper: 0.5) */
} ppow_params;

/* Output buffers, all device memory owned by the caller.  Any pointer except accepted_len may be
 * NULL, meaning "do not write this output".  Positions t >= valid_len[n] receive 0 in every
 * per-position output; a window with valid_len[n] == 0 receives 0 in every output. */
typedef struct {
    uint8_t *accept_flag;    /* [N,K] result of the per-position acceptance test (not prefix-ANDed) */
    int32_t *accepted_len;   /* [N]   k = number of leading accepted positions (App. C.1, tau) */
    float *reward_speedup;   /* [N]   k/(k*c + 1)                                  (Sec. 4.3.1) */
    float *reward_dist;      /* [N]   eta * 1[k = 0] * 1[Delta < eps]               (Sec. 4.3.2) */
    float *reward;           /* [N]   reward_speedup + reward_dist                  (Alg. 1, total reward) */
    float *delta;            /* [N]   proximity gap Delta (see ref_logp below)      (Sec. 4.3.2) */
    float *score;            /* [N]   s = mean over valid positions of crit         (Sec. 4.2, s_j) */
    float *kl;               /* [N,K] KL(P_t || Q_t), nats                          (Sec. 4.2) */
    float *conf;             /* [N,K] C(P_t) = 1 - H(P_t)/ln V, clamped to [0,1]    (Sec. 4.2) */
    float *crit;             /* [N,K] v_t = C(P_t) * KL(P_t || Q_t)                 (Sec. 4.2; Alg. 1) */
    float *logp_tok;         /* [N,K] log P_t(yhat_t); -inf for an out-of-range token */
    float *logq_tok;         /* [N,K] log Q_t(yhat_t); -inf for an out-of-range token */
    int32_t *target_argmax;  /* [N,K] argmax_v of the stored target logits, lowest index on ties */
    /* training-side quantities; asking for kl_rev or kl_rev_mean adds one fused multiply-add per logit pair */
    float *kl_rev;           /* [N,K] KL(Q_t || P_t), nats: the target-anchored regulariser's token-wise term
                                      (Sec. 4.1 objective; App. A.2) */
    float *kl_rev_mean;      /* [N]   its mean over the valid positions of the window (App. A.2) */
    float *nabla;            /* [N,K] alignment divergence exp(d) - d - 1, d = log P_t(yhat_t) - log Q_t(yhat_t)
                                      (App. E); +inf for an out-of-range token */
    float *lse_p;            /* [N,K] log sum_v exp(target/T), the softmax normaliser of P_t (Sec. 4.2) */
    float *lse_q;            /* [N,K] log sum_v exp(draft/T), that of Q_t; both are inputs of ppow_expected_acceptance */
} ppow_outputs;

/* Bytes of device scratch ppow_score_windows needs for these parameters (0 on invalid params). */
size_t ppow_score_workspace_bytes(const ppow_params *params);

/*
 * Scoring pass (Sec. 4.2 criticality, App. C.1 verification, Sec. 4.3 rewards; the criticality,
 * verification, proximity-gap and reward steps of Alg. 1).
 *
 *   draft_logits, target_logits  device, [N,K,V] of params->dtype (float32, bfloat16 or IEEE float16),
 *                                contiguous, aligned to their element size.  Both tensors are read from HBM
 *                                exactly once, in aligned 16-byte units: when V is not a multiple of the logits
 *                                per unit, or a base pointer is off a 16-byte boundary, the units that hold a
 *                                row's first and last logit are read whole (the neighbours' logits in them are
 *                                masked out), so up to 15 bytes before the first and after the last logit of a
 *                                tensor are read too -- bytes of the same aligned 16-byte unit as valid data.
 *                                Full speed needs both tensors at the same offset within a unit (any offset);
 *                                otherwise a slower scalar kernel runs.
 *   draft_tokens                 device, [N,K] int32.  A token outside [0,V) is rejected, gets
 *                                logp_tok = logq_tok = -inf, and sets PPOW_FLAG_TOKEN_RANGE.
 *   uniforms                     device, [N,K] float32 in [0,1), drawn by the caller;
 *                                may be NULL iff mode == PPOW_GREEDY.
 *   valid_len                    device, [N] int32 in [0,K], or NULL for "all K positions valid".
 *                                Positions t >= valid_len[n] are neither read nor scored.
 *   ref_logp                     device, [N] float32, or NULL.  If given, it is the target's
 *                                log-probability of its own reference window and
 *                                Delta = ref_logp[n] - sum_t log P_t(yhat_t).  If NULL,
 *                                Delta = sum_t [max_v log P_t(v) - log P_t(yhat_t)], the reference
 *                                token at each position taken from the same target logits.
 *   out                          host pointer to a struct of device pointers (read during the call).
 *   workspace                    device, >= ppow_score_workspace_bytes(params), 256-byte aligned.
 *                                Contents are undefined afterwards except the error word.
 *
 * Returns PPOW_OK once the work is enqueued.  N == 0 is a valid no-op.
 * If the error word afterwards carries PPOW_FLAG_DEVICE_TIMEOUT (ppow_read_error_flags returns
 * PPOW_ERR_DEVICE_TIMEOUT), a warp gave up on a bounded wait and left its work items unreduced: every output of
 * that call is undefined and must be discarded.
 */
ppow_status ppow_score_windows(const ppow_params *params,
                               const void *draft_logits, const void *target_logits,
                               const int32_t *draft_tokens, const float *uniforms,
                               const int32_t *valid_len, const float *ref_logp,
                               const ppow_outputs *out,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Same call, with two optional cudaEvent_t handles (NULL = none) that the library records on
 * `cuda_stream` immediately before and immediately after the row-reduction kernel, the one step of
 * the pass that streams the logits (Sec. 4.2 softmax/entropy/KL sums).  Lets a caller time that
 * kernel alone; the events stay owned by the caller. */
ppow_status ppow_score_windows_traced(const ppow_params *params,
                                      const void *draft_logits, const void *target_logits,
                                      const int32_t *draft_tokens, const float *uniforms,
                                      const int32_t *valid_len, const float *ref_logp,
                                      const ppow_outputs *out,
                                      void *workspace, size_t workspace_bytes, void *cuda_stream,
                                      void *event_reduce_begin, void *event_reduce_end);

/*
 * ppow_score_windows without a workspace argument.  (An addition of this library; the paper has
 * no counterpart.)  For callers that cannot obtain device scratch memory: code that runs beside a
 * framework which already owns all device memory and whose allocator it cannot reach, or code
 * that must not allocate after start-up.  The scratch is a fixed array of
 * ppow_noalloc_scratch_bytes() (4 MiB) of device global memory inside the library image; every GPU
 * that loads the library holds it until the process exits.  Inputs, outputs, stream and results
 * are exactly those of ppow_score_windows.  No memory is allocated or freed by this call.
 *   - Returns PPOW_ERR_UNSUPPORTED, launching nothing, when
 *     ppow_score_workspace_bytes(params) > ppow_noalloc_scratch_bytes().
 *   - All calls on one device share the array, and it keeps the previous call's contents; the work
 *     counter and error word that must start at zero are cleared on the stream by every call.
 *     Calls that overlap on the GPU (other streams or host threads) race on it: serialise them.
 *   - The first call on each device looks up the array's device address, which may load the
 *     module: make that first call outside any stream capture.
 *   - The address is remembered per device for the life of the process; do not use this entry point on a
 *     device whose context the process has destroyed (cudaDeviceReset) since the first call.
 *   - The error word of the call (out-of-range token, device-side timeout) sits in the shared array: read it
 *     with ppow_noalloc_read_error_flags (same semantics as ppow_read_error_flags; synchronises the stream)
 *     before the next call on the device clears it.
 */
size_t ppow_noalloc_scratch_bytes(void);
ppow_status ppow_noalloc_read_error_flags(uint32_t *flags_host, void *cuda_stream);
ppow_status ppow_score_windows_noalloc(const ppow_params *params,
                                       const void *draft_logits, const void *target_logits,
                                       const int32_t *draft_tokens, const float *uniforms,
                                       const int32_t *valid_len, const float *ref_logp,
                                       const ppow_outputs *out, void *cuda_stream);

/*
 * Group-relative advantage (Sec. 4.1): for every contiguous group of `group_size` windows (one rollout
 * group: G_roll drafts of the same prefix; the paper uses 8),
 *     advantage[i] = (reward[i] - mu) / (sigma + delta)
 * with mu and sigma the mean and the population standard deviation (divisor G) of the group's rewards
 * and delta >= 0 the stabiliser.  Computed in float64, stored as float32.
 *   reward, advantage   device, [N] float32 (may not alias)
 * Requires N >= 0, 1 <= group_size <= 1024 and N a multiple of group_size.  No workspace.
 */
ppow_status ppow_group_advantage(const float *reward, int32_t N, int32_t group_size, float delta,
                                 float *advantage, void *cuda_stream);

/*
 * Sequence form of Adaptive Divergence-Aware Windowing (Sec. 4.2; the window-selection step of Alg. 1):
 * for B responses stored back to back, response b owning positions [seq_offsets[b], seq_offsets[b+1]) of
 * `crit` (the per-position criticality v_t, e.g. the crit output of ppow_score_windows), computes for every
 * start j with a full window inside the response
 *     scores[seq_offsets[b] + j] = (1/K) * sum_{t=j}^{j+K-1} v_t          (s_j)
 * (0 at the last K-1 positions of a response, where no window starts), and draws one start per response
 * with probability s_j / sum_i s_i by inverse CDF from the caller's uniform u_b in [0,1): the first j whose
 * running sum of s exceeds u_b * sum_i s_i.  A response whose scores are all 0 draws floor(u_b * n_b)
 * (uniform); a response shorter than K has no start (-1).  Sums run in float64 in index order.
 *   crit          device, [seq_offsets[B]] float32, values >= 0
 *   seq_offsets   device, [B+1] int32, non-decreasing, seq_offsets[0] = 0
 *   scores        device, same length as crit, or NULL
 *   uniforms      device, [B] float32, or NULL iff starts is NULL
 *   starts        device, [B] int32 (start index relative to its response), or NULL
 * Requires B >= 0 and 1 <= K <= 1024.  No workspace.  One thread block per response.
 */
ppow_status ppow_sequence_windows(const float *crit, const int32_t *seq_offsets, int32_t B, int32_t K,
                                  float *scores, const float *uniforms, int32_t *starts, void *cuda_stream);

/*
 * ppow_sequence_windows under the hard-window curriculum (App. A, training configuration: the proportion of
 * ADAW-selected hard windows starts small and is raised over training, 0.2 / 0.4 / 0.6 in the paper's table;
 * the ablation without ADAW draws windows uniformly).  Scores are as above.  Each response b takes the ADAW
 * draw (proportional to s_j, from uniforms_draw[b]) iff uniforms_mix[b] < hard_frac, and otherwise the uniform
 * start floor(uniforms_draw[b] * n_b), n_b = number of starts with a full window.  hard_frac = 1 reproduces
 * ppow_sequence_windows, hard_frac = 0 is uniform window sampling.  The schedule of hard_frac over training
 * steps is the caller's.
 *   hard_frac       in [0,1] (else PPOW_ERR_INVALID_ARG)
 *   uniforms_mix    device, [B] float32 in [0,1): the per-response coin; required iff starts is given
 *   uniforms_draw   device, [B] float32 in [0,1): the draw within the chosen branch; required iff starts is given
 * Everything else as for ppow_sequence_windows.
 */
ppow_status ppow_sequence_windows_mixed(const float *crit, const int32_t *seq_offsets, int32_t B, int32_t K,
                                        float hard_frac, float *scores, const float *uniforms_mix,
                                        const float *uniforms_draw, int32_t *starts, void *cuda_stream);

/*
 * Expected acceptance probability per position (App. B.1): sum_v min(P_t(v), Q_t(v)) = 1 - TV(P_t, Q_t),
 * the probability that a token drafted from Q_t passes verification.  A second streaming pass over both
 * logit tensors that needs the softmax normalisers of the first: lse_p, lse_q as written by
 * ppow_score_windows (same params, same tensors).
 *   draft_logits, target_logits, valid_len   as for ppow_score_windows
 *   lse_p, lse_q       device, [N,K] float32
 *   expected_accept    device, [N,K] float32; 0 at positions t >= valid_len[n]
 * No workspace.
 */
ppow_status ppow_expected_acceptance(const ppow_params *params,
                                     const void *draft_logits, const void *target_logits,
                                     const int32_t *valid_len, const float *lse_p, const float *lse_q,
                                     float *expected_accept, void *cuda_stream);

/*
 * Log-probability of the target-preferred reference window (Sec. 4.3.2): the reference window is built
 * greedily by the target under its own prefix, y_t = argmax_v pi_target(v | x, y_<t).  Given the target's
 * logits along that window,
 *     ref_logp[n] = sum_{t < valid_len[n]} max_v log softmax(ref_target_logits[n,t,:] / T)(v),
 * which is what ppow_score_windows takes as `ref_logp` to evaluate the proximity gap Delta in its exact
 * form.  One more streaming pass over one [N,K,V] tensor (params->N, K, V, dtype, temperature are used).
 *   ref_target_logits   device, [N,K,V] of params->dtype, contiguous
 *   valid_len           device, [N] int32 or NULL, as for ppow_score_windows
 *   row_logp            device, [N,K] float32, required: max_v log softmax(...)(v) per position (0 at
 *                       positions t >= valid_len[n])
 *   ref_logp            device, [N] float32 or NULL: the window sums, added in position order (0 for an
 *                       empty window)
 * No workspace beyond row_logp.  One thread block per position.
 */
ppow_status ppow_reference_logprob(const ppow_params *params, const void *ref_target_logits,
                                   const int32_t *valid_len, float *row_logp, float *ref_logp, void *cuda_stream);

/* Copies the error word that the last ppow_score_windows call on `workspace` left behind into
 * *flags_host (PPOW_FLAG_* bits) and synchronises `cuda_stream` to do so.  Returns
 * PPOW_ERR_DEVICE_TIMEOUT if that bit is set, PPOW_ERR_CUDA on a CUDA failure, else PPOW_OK. */
ppow_status ppow_read_error_flags(const void *workspace, uint32_t *flags_host, void *cuda_stream);

/*
 * Self-test of the device-side failure report.  The scoring kernel's only waits are bounded waits on the
 * mbarriers of its copy pipeline; when one runs out the kernel sets PPOW_FLAG_DEVICE_TIMEOUT in the
 * workspace's error word and returns instead of hanging.  This call makes exactly that happen on purpose
 * and harmlessly: one warp waits, with the same bounded wait, on an mbarrier that nothing completes, for at
 * most `probes` probes (1..65536), and reports the same way.  Afterwards ppow_read_error_flags(workspace)
 * returns PPOW_ERR_DEVICE_TIMEOUT with that bit set; the context stays usable.
 *   workspace   device, >= 256 bytes, 256-byte aligned (its error word is cleared first)
 */
ppow_status ppow_selftest_wait_timeout(void *workspace, size_t workspace_bytes, uint32_t probes, void *cuda_stream);

/* Bytes of device scratch ppow_select_windows needs for N scores (0 if N <= 0). */
size_t ppow_select_workspace_bytes(int32_t N);

/*
 * ADAW window selection (Sec. 4.2: windows with larger s_j are prioritised): writes the indices
 * of the n_keep largest scores ordered by (score descending, index ascending); equal scores keep
 * the lower index first, and -0.0 ranks equal to +0.0.  Scores must not be NaN.
 *
 *   score      device, [N] float32
 *   selected   device, [n_keep] int32
 *   mask       device, [N] uint8 (1 = selected) or NULL
 *   workspace  device, >= ppow_select_workspace_bytes(N), 256-byte aligned
 * Requires 0 <= n_keep <= N <= 2^24.  n_keep == 0 or N == 0 is a valid no-op (mask is cleared).
 */
ppow_status ppow_select_windows(const float *score, int32_t N, int32_t n_keep,
                                int32_t *selected, uint8_t *mask,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The whole pass for callers whose buffers are in HOST memory (the steps of Alg. 1 from the criticality
 * score to the reward, followed by the ADAW ranking of Sec. 4.2): stages the windows
 * through `device_scratch` in chunks of as many windows as fit, scores each chunk, keeps the window
 * scores on the device, selects the n_keep best of all N windows and copies every requested result
 * back.  Same arguments as ppow_score_windows + ppow_select_windows except:
 *   - every input pointer, every pointer inside *out_host, selected_host [n_keep] and mask_host [N]
 *     (may be NULL) are host pointers; pinned memory lets the copies run asynchronously;
 *   - device_scratch is device memory, 256-byte aligned, of at least
 *     ppow_host_scratch_bytes(params, 1) bytes; ppow_host_scratch_bytes(params, N) avoids chunking.
 * Of *out_host, the outputs from accept_flag to target_argmax are served; the training-side ones
 * after them (kl_rev, kl_rev_mean, nabla, lse_p, lse_q) are ignored by this entry point.
 * All copies and kernels are enqueued on `cuda_stream`; results are valid once it has been
 * synchronised.  The token-range error flag is not reported by this entry point (an out-of-range
 * token still shows as logp_tok = -inf and a rejected position).
 */
size_t ppow_host_scratch_bytes(const ppow_params *params, int32_t chunk_windows);
ppow_status ppow_score_and_select_host(const ppow_params *params,
                                       const void *draft_logits, const void *target_logits,
                                       const int32_t *draft_tokens, const float *uniforms,
                                       const int32_t *valid_len, const float *ref_logp,
                                       const ppow_outputs *out_host,
                                       int32_t n_keep, int32_t *selected_host, uint8_t *mask_host,
                                       void *device_scratch, size_t scratch_bytes, void *cuda_stream);

/*
 * Measurement aid (an addition of this library; the paper has no counterpart): one read-only streaming pass
 * over `bytes` of device memory with 16-byte loads, XOR-folding every 32-bit word into *checksum.  Timed with
 * events around the call it gives the bandwidth a kernel that only reads reaches on this GPU, the ceiling the
 * scoring pass (which reads both logit tensors once and writes next to nothing) is compared with.
 *   data       device, 16-byte aligned; bytes a non-zero multiple of 16
 *   checksum   device, one uint32 (cleared on the stream, then written)
 */
ppow_status ppow_stream_read_probe(const void *data, size_t bytes, uint32_t *checksum, void *cuda_stream);

/* Number of kernels one ppow_score_windows call with these parameters launches (1: small problems are scored
 * in a single launch; 2: row reduction + window scan; 0 on invalid parameters).  Launch accounting only. */
int ppow_score_kernel_launches(const ppow_params *params);

/*
 * Bounds-checked build (an addition of this library; the paper has no counterpart).  The build script also
 * produces libppow_checked.so, the same sources compiled with -DPPOW_CHECKED: every index a kernel derives
 * from N, K, V, the valid lengths, a work item, a tile, a pipeline stage or a token id is tested before use;
 * a failing test never traps -- it is counted, the access is skipped, and PPOW_FLAG_BOUNDS is set in the
 * call's error word where there is one.  This call synchronises the device and returns the number of failed
 * checks since the library was loaded and the site code of the first one (1xx row reduction, 2xx window
 * scan, 3xx selection, 4xx training side).  In the ordinary library it writes zeros and returns
 * PPOW_ERR_UNSUPPORTED.
 *   failures_host     host, required        first_site_host   host or NULL
 */
ppow_status ppow_checked_failures(uint32_t *failures_host, uint32_t *first_site_host);

/*
 * Timeline build (an addition of this library; the paper has no counterpart).  The build script can also
 * produce libppow_timeline.so (-DPPOW_TIMELINE), in which every warp of the bulk-copy row kernel records eleven
 * 64-bit words per launch: start, first data arrival and end (global timer, ns), items and tiles it processed,
 * its SM, cycles spent waiting for copies, cycles spent in item ends, its total cycles, and the item-end cycles
 * up to the end of the warp reduction and from there to the opening of the next item.  This call
 * synchronises the device and copies the records of warps 0 .. warps-1 (at most 4096; warp = block * 8 + warp
 * in block) of the last launch to words_host[warps * 11].  `python -m paper_2605_14978_b200.timeline` prints a
 * summary.  In the ordinary library: PPOW_ERR_UNSUPPORTED.
 */
ppow_status ppow_timeline_read(uint64_t *words_host, size_t warps);

/* Static, never-NULL description of a status code. */
const char *ppow_status_string(ppow_status status);

/* Library version as major*10000 + minor*100 + patch. */
int ppow_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PPOW_H_ */
