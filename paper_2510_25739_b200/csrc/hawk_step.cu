// hawk_verify_step_host: one whole verify step driven from HOST buffers.
// Copies the step's inputs to caller-provided device staging, runs the three stages on the stream
// and copies the two result vectors back; nothing here computes anything itself.
#include "hawk_common.cuh"

extern "C" hawk_status hawk_verify_step_host(const hawk_step_host_args *a, hawk_stream_t stream)
{
    if (!a) return HAWK_ERR_NULL;
    if (a->B < 0 || a->K < 0 || a->H < 0 || a->D < 0 || a->V < 0) return HAWK_ERR_SHAPE;
    if (a->B == 0) return HAWK_OK;
    if (!a->h_q || !a->h_x || !a->h_q_probs || !a->h_draft || !a->h_u_accept || !a->h_u_resample ||
        !a->h_accept_len || !a->h_out_token)
        return HAWK_ERR_NULL;
    if (!a->d_q || !a->d_x || !a->d_q_probs || !a->d_draft || !a->d_u_accept || !a->d_u_resample || !a->d_attn_out ||
        !a->d_logits || !a->d_accept_len || !a->d_out_token || !a->d_k_cache || !a->d_v_cache || !a->d_prefix_len ||
        !a->d_w)
        return HAWK_ERR_NULL;
    const int S = 2 * a->B, M = S * a->K;
    const size_t hidden = static_cast<size_t>(a->H) * a->D;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    struct Copy {
        void *dst;
        const void *src;
        size_t bytes;
    } in[] = {
        {a->d_q, a->h_q, static_cast<size_t>(M) * hidden * 2},
        {a->d_x, a->h_x, static_cast<size_t>(M) * hidden * 2},
        {a->d_q_probs, a->h_q_probs, static_cast<size_t>(a->B) * a->K * a->V * 4},
        {a->d_draft, a->h_draft, static_cast<size_t>(a->B) * a->K * 4},
        {a->d_u_accept, a->h_u_accept, static_cast<size_t>(a->B) * a->K * 4},
        {a->d_u_resample, a->h_u_resample, static_cast<size_t>(a->B) * (a->K + 1) * 4},
    };
    for (const Copy &c : in)
        if (cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return HAWK_ERR_CUDA;

    hawk_status rc = hawk_verify_attn(a->d_q, a->d_k_cache, a->d_v_cache, a->d_prefix_len, a->d_attn_out, S, a->K, a->H,
                                      a->H_kv, a->D, a->L_cap, a->max_prefix_len, a->sm_scale, a->d_attn_workspace,
                                      a->attn_workspace_bytes, a->d_status, stream);
    if (rc != HAWK_OK) return rc;
    rc = hawk_head_proj(a->d_x, a->d_w, a->d_logits, M, static_cast<int>(hidden), a->V, a->v_begin, a->v_end,
                        a->d_status, stream);
    if (rc != HAWK_OK) return rc;
    rc = hawk_cfg_accept(a->d_logits, a->d_q_probs, a->d_draft, a->d_u_accept, a->d_u_resample, a->B, a->K, a->V,
                         a->v_begin, a->v_end, a->cfg_scale, a->temperature, a->top_k, 0, a->d_accept_len,
                         a->d_out_token, nullptr, a->d_accept_workspace, a->accept_workspace_bytes, a->d_status, stream);
    if (rc != HAWK_OK) return rc;
    if (cudaMemcpyAsync(a->h_accept_len, a->d_accept_len, static_cast<size_t>(a->B) * 4, cudaMemcpyDeviceToHost, st) !=
            cudaSuccess ||
        cudaMemcpyAsync(a->h_out_token, a->d_out_token, static_cast<size_t>(a->B) * 4, cudaMemcpyDeviceToHost, st) !=
            cudaSuccess)
        return HAWK_ERR_CUDA;
    return HAWK_OK;
}
