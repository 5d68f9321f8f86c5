#include "btc_internal.cuh"
namespace btc {
int launch_transform(const void *, int, const btc_transform &, void *, int, int, cudaStream_t) { return BTC_ERR_UNSUPPORTED; }
}
