#include "internal.h"
namespace m2rnn {
cudaError_t launch_bwd_bf16(const ScanArgs &, cudaStream_t) { return cudaErrorNotSupported; }
}
