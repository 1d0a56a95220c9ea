// hawk_verify_step_host: one whole verify step driven from HOST buffers.
// Copies the step's inputs to caller-provided device staging, runs the three stages on the stream
// and copies the two result vectors back; nothing here computes anything itself.
//
// The inputs that only the accept stage reads (the draft distributions are 85 % of a step's host
// bytes) travel on a second, library-owned stream while attention and the head projection run, and
// join the caller's stream before the accept stage: the step costs max(copies, kernels) instead of
// their sum.  The fork and join are event dependencies, so the call stays asynchronous and can be
// captured in a CUDA graph like any other stream work.
//
// Argument errors are found before anything is queued: the three stages' host-side checks run first,
// on the staging pointers and sizes the stages will be given, so a refused call leaves the stream, the
// staging buffers and the outputs as they were.
//
// State: the first call on a device creates one non-blocking stream and two events for it and keeps
// them for the life of the process (no device memory).  They are shared by every call on that
// device, so the queuing part of a call runs under a per-device mutex: calls from several host
// threads are queued one after the other, and the late copies of concurrent steps share the one side
// stream (they still overlap with kernels, not with each other).
#include <mutex>

#include "hawk_common.cuh"

namespace {

struct SideLane {
    std::mutex mu;  // held while a call queues its work: the fork/join events are recorded and waited on in pairs
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};

constexpr int kMaxDevices = 64;
SideLane g_lanes[kMaxDevices];

// The lane of the current device; its stream and events are created on the first call on that device
// (make that call outside stream capture).  Call with the lane's mutex NOT held; returns it unlocked.
SideLane *side_lane()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    SideLane &l = g_lanes[dev];
    std::lock_guard<std::mutex> lock(l.mu);
    if (!l.stream) {
        cudaStream_t st = nullptr;
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&e0, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) != cudaSuccess)
            return nullptr;
        l.stream = st;
        l.fork = e0;
        l.join = e1;
    }
    return &l;
}

}  // namespace

extern "C" hawk_status hawk_verify_step_host(const hawk_step_host_args *a, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_verify_step_host");
    if (!a) return HAWK_ERR_NULL;
    if (a->B < 0 || a->K < 0 || a->H < 0 || a->H_kv < 0 || a->D < 0 || a->V < 0 || a->L_cap < 0 ||
        a->max_prefix_len < 0)
        return HAWK_ERR_SHAPE;
    if (a->B == 0) return HAWK_OK;
    if (a->B > (1 << 20) || a->K > 64 || a->H > (1 << 16) || a->D > 1024) return HAWK_ERR_UNSUPPORTED;  // sizes below stay in range
    if (!a->h_q || !a->h_x || !a->h_q_probs || !a->h_draft || !a->h_u_accept || !a->h_u_resample ||
        !a->h_accept_len || !a->h_out_token)
        return HAWK_ERR_NULL;
    if (!a->d_q || !a->d_x || !a->d_q_probs || !a->d_draft || !a->d_u_accept || !a->d_u_resample || !a->d_attn_out ||
        !a->d_logits || !a->d_accept_len || !a->d_out_token || !a->d_k_cache || !a->d_v_cache || !a->d_prefix_len ||
        !a->d_w)
        return HAWK_ERR_NULL;
    const int S = 2 * a->B, M = S * a->K;
    const size_t hidden = static_cast<size_t>(a->H) * a->D;
    // every stage's argument checks, before anything is queued
    hawk_status rc = hawk_host::check_verify_attn_args(a->d_q, a->d_k_cache, a->d_v_cache, a->d_prefix_len, a->d_attn_out, S,
                                                       a->K, a->H, a->H_kv, a->D, a->L_cap, a->max_prefix_len, a->sm_scale,
                                                       a->d_attn_workspace, a->attn_workspace_bytes);
    if (rc != HAWK_OK) return rc;
    rc = hawk_host::check_head_proj_args(a->d_x, a->d_w, a->d_logits, M, static_cast<int>(hidden), a->V, a->v_begin,
                                         a->v_end);
    if (rc != HAWK_OK) return rc;
    rc = hawk_host::check_cfg_accept_args(a->d_logits, a->d_q_probs, a->d_draft, a->d_u_accept, a->d_u_resample, a->B, a->K,
                                          a->V, a->v_begin, a->v_end, a->cfg_scale, a->temperature, a->d_accept_len,
                                          a->d_out_token, nullptr, a->d_accept_workspace, a->accept_workspace_bytes);
    if (rc != HAWK_OK) return rc;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    struct Copy {
        void *dst;
        const void *src;
        size_t bytes;
    };
    // needed by attention and the head projection: on the caller's stream, first
    const Copy early[] = {
        {a->d_q, a->h_q, static_cast<size_t>(M) * hidden * 2},
        {a->d_x, a->h_x, static_cast<size_t>(M) * hidden * 2},
    };
    // needed by the accept stage only: on the side stream, behind everything queued on `stream` so far
    const Copy late[] = {
        {a->d_q_probs, a->h_q_probs, static_cast<size_t>(a->B) * a->K * a->V * 4},
        {a->d_draft, a->h_draft, static_cast<size_t>(a->B) * a->K * 4},
        {a->d_u_accept, a->h_u_accept, static_cast<size_t>(a->B) * a->K * 4},
        {a->d_u_resample, a->h_u_resample, static_cast<size_t>(a->B) * (a->K + 1) * 4},
    };
    SideLane *lane = side_lane();
    if (!lane) return HAWK_ERR_CUDA;
    std::lock_guard<std::mutex> queue_lock(lane->mu);
    if (cudaEventRecord(lane->fork, st) != cudaSuccess || cudaStreamWaitEvent(lane->stream, lane->fork, 0) != cudaSuccess)
        return HAWK_ERR_CUDA;
    for (const Copy &c : early)
        if (cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return HAWK_ERR_CUDA;
    bool late_ok = true;
    for (const Copy &c : late)
        late_ok = late_ok && cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, lane->stream) == cudaSuccess;
    // the join is queued whatever happens below, so that a failed call never leaves the side stream forked
    // off a capturing stream
    const bool joined = cudaEventRecord(lane->join, lane->stream) == cudaSuccess;

    rc = hawk_verify_attn(a->d_q, a->d_k_cache, a->d_v_cache, a->d_prefix_len, a->d_attn_out, S, a->K, a->H,
                          a->H_kv, a->D, a->L_cap, a->max_prefix_len, a->sm_scale, a->d_attn_workspace,
                          a->attn_workspace_bytes, a->d_status, stream);
    if (rc == HAWK_OK)
        rc = hawk_head_proj(a->d_x, a->d_w, a->d_logits, M, static_cast<int>(hidden), a->V, a->v_begin, a->v_end,
                            a->d_status, stream);
    const bool rejoined = joined && cudaStreamWaitEvent(st, lane->join, 0) == cudaSuccess;
    if (rc != HAWK_OK) return rc;
    if (!rejoined || !late_ok) return HAWK_ERR_CUDA;
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
