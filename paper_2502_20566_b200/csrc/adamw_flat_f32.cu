// Instantiates the flat-buffer kernels for f32 gradients (one translation unit per gradient type
// so that the builds run in parallel).
#include "adamw_flat.cuh"

namespace sradamw {
template cudaError_t launch_adamw_flat_g<true>(uint16_t*, const void*, uint16_t*, uint16_t*, uint64_t, uint64_t, uint32_t,
                                              uint32_t, uint32_t, const PhiloxKeys&, const StepScalars&,
                                              const DeviceInfo&, cudaStream_t);
}  // namespace sradamw
