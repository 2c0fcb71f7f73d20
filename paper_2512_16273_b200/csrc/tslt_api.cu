// Version, status strings and the workspace status query of libtslt.
#include <cuda_runtime.h>

#include "../../include/tslt.h"

extern "C" int tslt_version(void) { return 100; }

extern "C" const char* tslt_status_string(int status) {
    switch (status) {
        case TSLT_OK: return "ok";
        case TSLT_ERR_INVALID_ARG: return "invalid argument";
        case TSLT_ERR_UNSUPPORTED: return "unsupported dtype, size or shape";
        case TSLT_ERR_WORKSPACE: return "workspace too small";
        case TSLT_ERR_CUDA: return "CUDA runtime error";
        case TSLT_ERR_DEVICE_STATUS: return "the device status word of the workspace is not zero; outputs of that call are invalid";
        case TSLT_ERR_STATIC_SCRATCH: return "problem needs more scratch than the array built into the library holds";
        default: return "unknown status";
    }
}

extern "C" int tslt_workspace_status(const void* workspace, void* stream, int* device_status) {
    if (!workspace) return TSLT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TSLT_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TSLT_ERR_CUDA;
    if (device_status) *device_status = word;
    return word == 0 ? TSLT_OK : TSLT_ERR_DEVICE_STATUS;
}
