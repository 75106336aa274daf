#include "internal.h"
namespace m2rnn {
// One decoding step = a T=1 scan whose initial and final state share storage.
cudaError_t launch_decode_bf16(const ScanArgs &a, cudaStream_t s) { return launch_fwd_bf16(a, s); }
}  // namespace m2rnn
