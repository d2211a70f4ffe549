// SwiGLU pair transition on tcgen05 (see fast.cuh).
#include "fast.cuh"

namespace ntp {

bool fast_transition_supported(int c, int hidden) { (void)c; (void)hidden; return false; }

nt_status fast_transition(void*, const nt_transition_weights*, float, int, int, long long, void*, int*, cudaStream_t) {
  return NT_ERR_UNSUPPORTED;
}

}  // namespace ntp
