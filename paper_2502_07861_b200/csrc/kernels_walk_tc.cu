// SoftmaxBalance (Algorithm 2) with the Gram tiles on the tensor cores (tcgen05 / TMEM / TMA).
#include "common.cuh"

namespace bkv {

bool walk_tc_supported(const Geom& G) { (void)G; return false; }

cudaError_t walk_tc_prepare(const Geom& G, const Arena& A, int64_t total_rows, void** tmaps_out) {
  (void)G; (void)A; (void)total_rows;
  *tmaps_out = nullptr;
  return cudaErrorNotSupported;
}

void walk_tc_release(void* tmaps) { (void)tmaps; }

cudaError_t launch_walk_tc(const Geom&, const Arena&, const CallDesc*, int, int, const CallStat*, const float*,
                           int8_t*, int8_t*, float*, float*, unsigned long long*, int*, const void*, const void*,
                           cudaStream_t) {
  return cudaErrorNotSupported;
}

}  // namespace bkv
