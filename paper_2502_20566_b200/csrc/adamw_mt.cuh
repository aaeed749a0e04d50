// Multi-tensor kernel of the fused SR-AdamW step and its launcher, for one gradient type.
#pragma once

#include "adamw_body.cuh"

namespace sradamw {

// Blocks walk the chunk table; a chunk is up to kMtChunkElems consecutive elements of one tensor.
// Element indices restart at 0 in every tensor and chunk starts are multiples of 8, so an aligned
// tensor is processed as whole noise groups.  MODE 1: reference arithmetic; 2 / 3: branch-free
// arithmetic without / with the gradient scale.  Tensors whose buffers are not 16-byte aligned go
// element by element.
template <bool G32, uint32_t FLAGS, int MODE>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocksPerSM)
k_sr_adamw_mt(const MtTensor* __restrict__ tensors, const MtChunk* __restrict__ chunks, uint32_t num_chunks,
              uint32_t tensor_id_base, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K,
              const __grid_constant__ StepScalars S) {
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    for (uint32_t c = blockIdx.x; c < num_chunks; c += gridDim.x) {
        const MtChunk ch = chunks[c];
        const MtTensor T = tensors[ch.tensor];
        const uint64_t start = static_cast<uint64_t>(ch.chunk) * kMtChunkElems;
        const uint64_t remaining = T.n - start;
        const uint32_t len = remaining < kMtChunkElems ? static_cast<uint32_t>(remaining) : kMtChunkElems;
        const uint32_t c2 = tensor_id_base + ch.tensor;
        if (T.vec_ok) {
            const uint32_t nvec = len >> 3;
            const uint64_t vec0 = start >> 3;
            const uint32_t c1 = static_cast<uint32_t>(start >> 33);   // a chunk never crosses a multiple of 2^33
            for (uint32_t j = threadIdx.x; j < nvec; j += blockDim.x) {
                const uint64_t idx0 = start + (static_cast<uint64_t>(j) << 3);
                if (MODE == 1)
                    step_vec8_reference<G32, FLAGS, true>(T.p, T.g, T.m, T.v, vec0 + j, idx0, c2, seed_hi, gscale, K, S);
                else
                    step_vec8_fast<G32, FLAGS, MODE == 3>(T.p, T.g, T.m, T.v, vec0 + j, idx0, c1, c2, seed_hi, gscale, K, S);
            }
            const uint32_t done = nvec << 3;
            if (threadIdx.x < len - done) {
                const uint64_t i = start + done + threadIdx.x;
                step_scalar<G32, FLAGS>(T.p, T.g, T.m, T.v, i, i, c2, seed_hi, gscale, K, S);
            }
        } else {
            for (uint32_t j = threadIdx.x; j < len; j += blockDim.x)
                step_scalar<G32, FLAGS>(T.p, T.g, T.m, T.v, start + j, start + j, c2, seed_hi, gscale, K, S);
        }
    }
}

template <bool G32, uint32_t FLAGS, int MODE>
cudaError_t launch_mt_mode(const MtTensor* tensors, const MtChunk* chunks, uint32_t num_chunks, uint32_t tensor_id_base,
                           uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev,
                           cudaStream_t stream) {
    auto k = k_sr_adamw_mt<G32, FLAGS, MODE>;
    const unsigned resident = static_cast<unsigned>(resident_blocks(k, dev));
    const unsigned grid = num_chunks < resident ? num_chunks : resident;
    k<<<grid, kBlockThreads, 0, stream>>>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S);
    return cudaGetLastError();
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_mt_flags(const MtTensor* tensors, const MtChunk* chunks, uint32_t num_chunks, uint32_t tensor_id_base,
                            uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev,
                            cudaStream_t stream) {
    if (!fast_path_allowed(S))
        return launch_mt_mode<G32, FLAGS, 1>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
    if (needs_scale(S))
        return launch_mt_mode<G32, FLAGS, 3>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
    return launch_mt_mode<G32, FLAGS, 2>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
}

template <bool G32>
cudaError_t launch_adamw_mt_g(const MtTensor* tensors, const MtChunk* chunks, uint32_t num_chunks,
                              uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                              const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
#define SR_MT(F) launch_mt_flags<G32, F>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream)
    SR_DISPATCH_FLAGS(SR_MT)
#undef SR_MT
}

}  // namespace sradamw
