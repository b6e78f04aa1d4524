// tcgen05 engine: placeholder until the tensor-core kernels land (every product goes to the FFMA engine).
#include "common.cuh"

namespace ulsnn {

static __device__ int g_dev_status;

bool tc_gemm_supported(const GemmDesc&) { return false; }
int tc_tile_m() { return 128; }
int tc_tile_n(const GemmDesc&) { return 256; }
ulsnn_status_t tc_gemm_launch(const GemmDesc&, bool, cudaStream_t) { return ULSNN_ERR_INVALID_ARG; }

ulsnn_status_t device_status_fetch_and_clear(cudaStream_t stream, int* word) {
    if (cudaStreamSynchronize(stream) != cudaSuccess) return ULSNN_ERR_CUDA;
    if (cudaMemcpyFromSymbol(word, g_dev_status, sizeof(int)) != cudaSuccess) return ULSNN_ERR_CUDA;
    if (*word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_dev_status, &zero, sizeof(int)) != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    return ULSNN_OK;
}

}  // namespace ulsnn
