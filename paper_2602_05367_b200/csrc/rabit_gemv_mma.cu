// placeholder until the integer-MMA GEMV lands
#include "rabit_internal.h"
bool rabit_gemv_mma_supports(const rabit_layer&, int) { return false; }
cudaError_t rabit_launch_gemv_mma(const rabit_layer&, const void*, void*, int, cudaStream_t) { return cudaErrorNotSupported; }
