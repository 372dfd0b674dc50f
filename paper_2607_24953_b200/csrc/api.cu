// Small host-side entry points of libfp4q: status strings, version, workspace handling.
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
