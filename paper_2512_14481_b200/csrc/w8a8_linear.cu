// Static W8A8 linear (placeholder until the tcgen05 kernel lands).
#include "common.cuh"

namespace sasq {
SASQ_DEFINE_STATUS_WORD(g_linear_status)
int linear_status_read_and_clear(cudaStream_t st) { return g_linear_status_read_and_clear(st); }
}  // namespace sasq

extern "C" {
size_t sasq_static_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K) { (void)T; (void)N; (void)K; return 0; }
int sasq_static_w8a8_linear(const void*, const int8_t*, const float*, const float*, const void*, void*, int32_t*,
                            int64_t, int64_t, int64_t, int, int, void*, size_t, void*) {
    return SASQ_ERR_UNSUPPORTED;
}
}
