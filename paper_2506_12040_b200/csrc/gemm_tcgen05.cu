#include "btc_internal.cuh"
namespace btc {
int launch_gemm_tcgen05(const LinearArgs &, cudaStream_t) { return BTC_ERR_UNSUPPORTED; }
size_t gemm_tcgen05_workspace_bytes(int, int, int, int, int) { return 0; }
}
