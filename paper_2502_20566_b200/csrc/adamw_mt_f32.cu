// Instantiates the multi-tensor kernels for f32 gradients.
#include "adamw_mt.cuh"

namespace sradamw {
template cudaError_t launch_adamw_mt_g<true>(const MtWork*, uint32_t, uint32_t, uint32_t, uint32_t,
                                            const PhiloxKeys&, const StepScalars&, const DeviceInfo&, cudaStream_t);
}  // namespace sradamw
