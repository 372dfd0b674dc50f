// Small host-side entry points of libfp4q: status strings, version, workspace handling.
#include <cstddef>

#include "common.cuh"

using namespace fp4q;

extern "C" const char *fp4q_status_string(fp4q_status s)
{
    switch (s) {
        case FP4Q_OK: return "ok";
        case FP4Q_ERR_NULL: return "a required pointer is NULL";
        case FP4Q_ERR_SHAPE: return "bad shape or leading dimension";
        case FP4Q_ERR_ALIGN: return "pointer or leading dimension is misaligned";
        case FP4Q_ERR_UNSUPPORTED: return "unsupported request";
        case FP4Q_ERR_WORKSPACE: return "workspace missing or too small";
        case FP4Q_ERR_CUDA: return "a CUDA call failed";
        case FP4Q_ERR_TIMEOUT: return "a bounded device-side wait expired";
    }
    return "unknown status";
}

extern "C" int fp4q_version(void) { return 100; }

extern "C" size_t fp4q_workspace_bytes(void) { return sizeof(Workspace); }

extern "C" fp4q_status fp4q_workspace_status(void *ws, void *stream)
{
    if (!ws) return FP4Q_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t host[2] = {0u, 0u};
    if (cudaMemcpyAsync(host, ws, sizeof host, cudaMemcpyDeviceToHost, s) != cudaSuccess) return FP4Q_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FP4Q_ERR_CUDA;
    if (host[0] == 0u) return FP4Q_OK;
    if (cudaMemsetAsync(ws, 0, sizeof host, s) != cudaSuccess) return FP4Q_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FP4Q_ERR_CUDA;
    return host[0] == (uint32_t)FP4Q_ERR_TIMEOUT ? FP4Q_ERR_TIMEOUT : FP4Q_ERR_CUDA;
}

// The two configuration words of a workspace (they persist until rewritten; fp4q_workspace_status clears only the status).
static fp4q_status set_workspace_word(void *ws, size_t offset, uint32_t value, void *stream)
{
    if (!ws) return FP4Q_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(static_cast<uint8_t *>(ws) + offset, &value, sizeof value, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return FP4Q_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;   // `value` lives on this stack frame
}

extern "C" fp4q_status fp4q_workspace_set_wait_limit(void *ws, uint32_t polls, void *stream)
{
    return set_workspace_word(ws, offsetof(Workspace, wait_limit), polls, stream);
}

extern "C" fp4q_status fp4q_debug_withhold_load(void *ws, uint32_t nth_load, void *stream)
{
    return set_workspace_word(ws, offsetof(Workspace, withhold_load), nth_load, stream);
}
