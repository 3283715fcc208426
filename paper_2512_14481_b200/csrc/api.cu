// Status strings, device checks and the sticky device status word.
#include "common.cuh"

namespace sasq {

int fakequant_status_read_and_clear(cudaStream_t st);
int linear_status_read_and_clear(cudaStream_t st);

int device_sm_count_if_sm100() {
    // cached per device ordinal; 0 = not queried yet, -1 = not sm_100
    static int cache[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cache[dev] != 0) return cache[dev];
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    cache[dev] = (major == 10 && sms > 0) ? sms : -1;
    return cache[dev];
}

}  // namespace sasq

extern "C" {

const char* sasq_status_string(int status) {
    switch (status) {
        case SASQ_OK: return "SASQ_OK";
        case SASQ_ERR_INVALID_ARG: return "SASQ_ERR_INVALID_ARG: null or misaligned pointer, bad size, dtype or bit-width";
        case SASQ_ERR_UNSUPPORTED: return "SASQ_ERR_UNSUPPORTED: shape constraint not met or device is not sm_100";
        case SASQ_ERR_WORKSPACE: return "SASQ_ERR_WORKSPACE: workspace missing, misaligned or too small";
        case SASQ_ERR_BAD_SCALE: return "SASQ_ERR_BAD_SCALE: a quantization factor is zero or not finite";
        case SASQ_ERR_TIMEOUT: return "SASQ_ERR_TIMEOUT: a bounded wait inside a kernel gave up";
        case SASQ_ERR_CUDA: return "SASQ_ERR_CUDA: a CUDA call failed";
        default: return "unknown SASQ status";
    }
}

int sasq_device_status(void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int a = sasq::fakequant_status_read_and_clear(st);
    const int b = sasq::linear_status_read_and_clear(st);
    return a > b ? a : b;
}

}  // extern "C"
