#include "launch.h"
#include "../../include/ue5m3.h"
namespace ue5m3 {
int launch_gemm(const GemmArgs&, int, cudaStream_t) { return UE5M3_ERR_UNSUPPORTED; }
int read_and_clear_device_status() { return cudaDeviceSynchronize() == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA; }
}
