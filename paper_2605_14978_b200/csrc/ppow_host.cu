// End-to-end entry point for callers whose buffers live in host memory: stages windows through a
// caller-provided device scratch buffer in chunks, scores each chunk with ppow_score_windows, keeps
// the window scores on the device, runs ppow_select_windows over all N of them and copies every
// result back.  Everything is enqueued on one stream; the library still allocates nothing.
#include "../../include/ppow.h"

#include <cuda_runtime.h>

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct ChunkLayout {
    size_t draft, target, tokens, uniforms, valid_len, ref_logp;
    size_t pos_u8, pos_f32[5], pos_i32, win_i32, win_f32[5];
    size_t workspace, workspace_bytes;
    size_t total;
};

// Device layout of one staged chunk of `cw` windows out of p->N.
ChunkLayout chunk_layout(const ppow_params *p, int32_t cw)
{
    ChunkLayout L;
    const size_t es = p->dtype == PPOW_F32 ? 4 : 2;
    const size_t rows = (size_t)cw * p->K;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.draft = take(rows * p->V * es);
    L.target = take(rows * p->V * es);
    L.tokens = take(rows * 4);
    L.uniforms = take(rows * 4);
    L.valid_len = take((size_t)cw * 4);
    L.ref_logp = take((size_t)cw * 4);
    L.pos_u8 = take(rows);
    for (int i = 0; i < 5; ++i) L.pos_f32[i] = take(rows * 4);
    L.pos_i32 = take(rows * 4);
    L.win_i32 = take((size_t)cw * 4);
    for (int i = 0; i < 5; ++i) L.win_f32[i] = take((size_t)cw * 4);
    // the workspace serves every chunk the loop will score: full chunks of cw windows and, when cw does not
    // divide N, a shorter last one -- whose work plan can be finer, hence larger, than a full chunk's
    ppow_params q = *p;
    q.N = cw;
    L.workspace_bytes = ppow_score_workspace_bytes(&q);
    const int32_t tail = p->N % cw;
    if (tail > 0) {
        q.N = tail;
        const size_t t = ppow_score_workspace_bytes(&q);
        if (t > L.workspace_bytes) L.workspace_bytes = t;
    }
    L.workspace = take(L.workspace_bytes);
    L.total = off;
    return L;
}

struct GlobalLayout {
    size_t score, selected, mask, select_ws, select_ws_bytes, chunk0;
};

GlobalLayout global_layout(const ppow_params *p)
{
    GlobalLayout G;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    G.score = take((size_t)p->N * 4);
    G.selected = take((size_t)p->N * 4);
    G.mask = take((size_t)p->N);
    G.select_ws_bytes = ppow_select_workspace_bytes(p->N);
    G.select_ws = take(G.select_ws_bytes);
    G.chunk0 = off;
    return G;
}

}  // namespace

extern "C" size_t ppow_host_scratch_bytes(const ppow_params *params, int32_t chunk_windows)
{
    if (!params || params->N <= 0 || chunk_windows <= 0) return 0;
    if (ppow_score_workspace_bytes(params) == 0) return 0;
    if (chunk_windows > params->N) chunk_windows = params->N;
    return global_layout(params).chunk0 + chunk_layout(params, chunk_windows).total;
}

extern "C" ppow_status ppow_score_and_select_host(const ppow_params *params,
                                                  const void *draft_logits, const void *target_logits,
                                                  const int32_t *draft_tokens, const float *uniforms,
                                                  const int32_t *valid_len, const float *ref_logp,
                                                  const ppow_outputs *out_host,
                                                  int32_t n_keep, int32_t *selected_host, uint8_t *mask_host,
                                                  void *device_scratch, size_t scratch_bytes, void *cuda_stream)
{
    if (!params || !out_host) return PPOW_ERR_INVALID_ARG;
    if (params->N == 0) return PPOW_OK;
    if (ppow_score_workspace_bytes(params) == 0)
        return params->K > 32 ? PPOW_ERR_UNSUPPORTED : PPOW_ERR_INVALID_ARG;
    if (!draft_logits || !target_logits || !draft_tokens || !out_host->accepted_len) return PPOW_ERR_INVALID_ARG;
    if (params->mode == PPOW_STOCHASTIC && !uniforms) return PPOW_ERR_INVALID_ARG;
    if (n_keep < 0 || n_keep > params->N || (n_keep > 0 && !selected_host)) return PPOW_ERR_INVALID_ARG;
    if (!device_scratch || ((uintptr_t)device_scratch % 256)) return PPOW_ERR_WORKSPACE;

    // largest chunk (in windows) that fits the scratch
    const GlobalLayout G = global_layout(params);
    int32_t cw = params->N;
    while (cw > 1 && G.chunk0 + chunk_layout(params, cw).total > scratch_bytes) cw = (cw + 1) / 2;
    if (G.chunk0 + chunk_layout(params, cw).total > scratch_bytes) return PPOW_ERR_WORKSPACE;
    const ChunkLayout L = chunk_layout(params, cw);

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char *base = (char *)device_scratch;
    char *cb = base + G.chunk0;
    const size_t es = params->dtype == PPOW_F32 ? 4 : 2;
    const int32_t K = params->K;
    const size_t row_bytes = (size_t)params->V * es;
    float *d_score = (float *)(base + G.score);

#define PPOW_COPY(dst, src, bytes, kind)                                                              \
    do {                                                                                              \
        if ((bytes) > 0 && cudaMemcpyAsync((dst), (src), (bytes), (kind), stream) != cudaSuccess)     \
            return PPOW_ERR_CUDA;                                                                     \
    } while (0)

    for (int32_t n0 = 0; n0 < params->N; n0 += cw) {
        const int32_t nw = (params->N - n0 < cw) ? (params->N - n0) : cw;
        const size_t rows = (size_t)nw * K, r0 = (size_t)n0 * K;
        PPOW_COPY(cb + L.draft, (const char *)draft_logits + r0 * row_bytes, rows * row_bytes, cudaMemcpyHostToDevice);
        PPOW_COPY(cb + L.target, (const char *)target_logits + r0 * row_bytes, rows * row_bytes, cudaMemcpyHostToDevice);
        PPOW_COPY(cb + L.tokens, draft_tokens + r0, rows * 4, cudaMemcpyHostToDevice);
        if (uniforms) PPOW_COPY(cb + L.uniforms, uniforms + r0, rows * 4, cudaMemcpyHostToDevice);
        if (valid_len) PPOW_COPY(cb + L.valid_len, valid_len + n0, (size_t)nw * 4, cudaMemcpyHostToDevice);
        if (ref_logp) PPOW_COPY(cb + L.ref_logp, ref_logp + n0, (size_t)nw * 4, cudaMemcpyHostToDevice);

        ppow_params q = *params;
        q.N = nw;
        ppow_outputs o = {};   // outputs this entry point does not stage (kl_rev, nabla, ...) stay NULL
        o.accept_flag = out_host->accept_flag ? (uint8_t *)(cb + L.pos_u8) : nullptr;
        o.kl = out_host->kl ? (float *)(cb + L.pos_f32[0]) : nullptr;
        o.conf = out_host->conf ? (float *)(cb + L.pos_f32[1]) : nullptr;
        o.crit = out_host->crit ? (float *)(cb + L.pos_f32[2]) : nullptr;
        o.logp_tok = out_host->logp_tok ? (float *)(cb + L.pos_f32[3]) : nullptr;
        o.logq_tok = out_host->logq_tok ? (float *)(cb + L.pos_f32[4]) : nullptr;
        o.target_argmax = out_host->target_argmax ? (int32_t *)(cb + L.pos_i32) : nullptr;
        o.accepted_len = (int32_t *)(cb + L.win_i32);
        o.reward_speedup = out_host->reward_speedup ? (float *)(cb + L.win_f32[0]) : nullptr;
        o.reward_dist = out_host->reward_dist ? (float *)(cb + L.win_f32[1]) : nullptr;
        o.reward = out_host->reward ? (float *)(cb + L.win_f32[2]) : nullptr;
        o.delta = out_host->delta ? (float *)(cb + L.win_f32[3]) : nullptr;
        o.score = d_score + n0;   // scores stay on the device for the selection
        const ppow_status st = ppow_score_windows(
            &q, cb + L.draft, cb + L.target, (const int32_t *)(cb + L.tokens),
            uniforms ? (const float *)(cb + L.uniforms) : nullptr,
            valid_len ? (const int32_t *)(cb + L.valid_len) : nullptr,
            ref_logp ? (const float *)(cb + L.ref_logp) : nullptr, &o, cb + L.workspace, L.workspace_bytes, stream);
        if (st != PPOW_OK) return st;

        if (o.accept_flag) PPOW_COPY(out_host->accept_flag + r0, o.accept_flag, rows, cudaMemcpyDeviceToHost);
        if (o.kl) PPOW_COPY(out_host->kl + r0, o.kl, rows * 4, cudaMemcpyDeviceToHost);
        if (o.conf) PPOW_COPY(out_host->conf + r0, o.conf, rows * 4, cudaMemcpyDeviceToHost);
        if (o.crit) PPOW_COPY(out_host->crit + r0, o.crit, rows * 4, cudaMemcpyDeviceToHost);
        if (o.logp_tok) PPOW_COPY(out_host->logp_tok + r0, o.logp_tok, rows * 4, cudaMemcpyDeviceToHost);
        if (o.logq_tok) PPOW_COPY(out_host->logq_tok + r0, o.logq_tok, rows * 4, cudaMemcpyDeviceToHost);
        if (o.target_argmax) PPOW_COPY(out_host->target_argmax + r0, o.target_argmax, rows * 4, cudaMemcpyDeviceToHost);
        PPOW_COPY(out_host->accepted_len + n0, o.accepted_len, (size_t)nw * 4, cudaMemcpyDeviceToHost);
        if (o.reward_speedup) PPOW_COPY(out_host->reward_speedup + n0, o.reward_speedup, (size_t)nw * 4, cudaMemcpyDeviceToHost);
        if (o.reward_dist) PPOW_COPY(out_host->reward_dist + n0, o.reward_dist, (size_t)nw * 4, cudaMemcpyDeviceToHost);
        if (o.reward) PPOW_COPY(out_host->reward + n0, o.reward, (size_t)nw * 4, cudaMemcpyDeviceToHost);
        if (o.delta) PPOW_COPY(out_host->delta + n0, o.delta, (size_t)nw * 4, cudaMemcpyDeviceToHost);
    }
    if (out_host->score) PPOW_COPY(out_host->score, d_score, (size_t)params->N * 4, cudaMemcpyDeviceToHost);

    int32_t *d_sel = (int32_t *)(base + G.selected);
    uint8_t *d_mask = mask_host ? (uint8_t *)(base + G.mask) : nullptr;
    const ppow_status st = ppow_select_windows(d_score, params->N, n_keep, d_sel, d_mask, base + G.select_ws,
                                               G.select_ws_bytes, stream);
    if (st != PPOW_OK) return st;
    if (n_keep > 0) PPOW_COPY(selected_host, d_sel, (size_t)n_keep * 4, cudaMemcpyDeviceToHost);
    if (mask_host) PPOW_COPY(mask_host, d_mask, (size_t)params->N, cudaMemcpyDeviceToHost);
#undef PPOW_COPY
    return PPOW_OK;
}
