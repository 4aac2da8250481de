// TF32 tensor-pipe rate probe (defined next to the tensor-core kernel, whose PTX helpers it uses).
#pragma once
#include <cuda_runtime.h>
#include "mom.h"
namespace mom {
mom_status_t tc_probe_tf32(double milliseconds, void *scratch, cudaStream_t stream, double *tflops);
}
