// Prefill attention over the prompt segment (paper Section 3.1 / 3.3: the prefill kernel is
// the special case of the customised SDPA kernel that sees only the query and the prompt
// key/value, batch-first in and out): causal self-attention of every prompt position,
//     out[b,i,h,:] = softmax_{j<=i}( q[b,i,h,:] . K[b,j,:] / sqrt(D) + bias ) . V[b,j,:],
// with K/V read from the prompt segment that segkv_prefill_write has just stored.
//
// Every supported head size (64, 128, 256) runs on the tcgen05 kernel of segkv_prefill_tc5.cu;
// this file is the entry the host API calls.
#include "segkv_internal.h"

namespace segkv_impl {

bool prefill_sdpa_supported(const Dims& d) { return prefill_tc5_supported(d); }

cudaError_t launch_prefill_sdpa(const Dims& d, const PrefillArgs& a, cudaStream_t st) {
    if (!prefill_tc5_supported(d)) return cudaErrorInvalidValue;
    return launch_prefill_tc5(d, a, st);
}

}  // namespace segkv_impl
