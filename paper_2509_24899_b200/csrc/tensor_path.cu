// Placeholder until the tcgen05 kernels land: the tensor path reports "not supported".
#include "as_internal.h"
cudaError_t as_tensor_init() { return cudaSuccess; }
cudaError_t as_tensor_kpass(const as_launch_args&, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t as_tensor_qpass(const as_launch_args&, cudaStream_t) { return cudaErrorNotSupported; }
