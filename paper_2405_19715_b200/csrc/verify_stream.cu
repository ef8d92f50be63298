// Streaming verify/correct kernel (placeholder until the persistent TMA kernel lands).
#include "specdec_internal.h"

bool verify_stream_supported(const VerifyParams&, specdec_dtype) { return false; }

cudaError_t launch_verify_stream(const VerifyParams&, specdec_dtype, int, cudaStream_t, int* n_launch) {
    *n_launch = 0;
    return cudaErrorNotSupported;
}
