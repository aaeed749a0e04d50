// Flat-buffer kernel of the fused SR-AdamW step and its launcher, for one gradient type.
#pragma once

#include "adamw_body.cuh"

namespace sradamw {

// MODE 0: element-wise (any alignment, any offset)
//      1: 16-byte vectors, reference arithmetic, per-element noise (elem_offset not a multiple of 8)
//      2: 16-byte vectors, branch-free arithmetic, gradient used as is
//      3: 16-byte vectors, branch-free arithmetic, gradient multiplied by gscale
// Persistent grid: thread t takes vectors t, t + T, t + 2T, ... (T = threads in the grid).
// For modes 2 and 3 every index of the launch has the same (index >> 33) = c1.
template <bool G32, uint32_t FLAGS, int MODE>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocksPerSM)
k_sr_adamw_flat(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset, uint32_t c1,
                uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K,
                const __grid_constant__ StepScalars S) {
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    if (MODE == 0) {
        for (uint64_t i = tid; i < n; i += stride)
            step_scalar<G32, FLAGS>(p, g, m, v, i, elem_offset + i, tensor_id, seed_hi, gscale, K, S);
        return;
    }
    const uint64_t nvec = n >> 3;
    for (uint64_t vec = tid; vec < nvec; vec += stride) {
        const uint64_t idx0 = elem_offset + (vec << 3);
        if (MODE == 1)
            step_vec8_reference<G32, FLAGS, false>(p, g, m, v, vec, idx0, tensor_id, seed_hi, gscale, K, S);
        else
            step_vec8_fast<G32, FLAGS, MODE == 3>(p, g, m, v, vec, idx0, c1, tensor_id, seed_hi, gscale, K, S);
    }
    const uint64_t done = nvec << 3;
    if (tid < n - done)
        step_scalar<G32, FLAGS>(p, g, m, v, done + tid, elem_offset + done + tid, tensor_id, seed_hi, gscale, K, S);
}

template <bool G32, uint32_t FLAGS, int MODE>
cudaError_t launch_flat_mode(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                             uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S,
                             const DeviceInfo& dev, cudaStream_t stream) {
    auto k = k_sr_adamw_flat<G32, FLAGS, MODE>;
    const uint64_t items = MODE == 0 ? n : (n >> 3) + 8;   // + 8: enough threads for the ragged tail
    k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(p, g, m, v, n, elem_offset,
                                                             static_cast<uint32_t>(elem_offset >> 33), tensor_id,
                                                             seed_hi, K, S);
    return cudaGetLastError();
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_flat_flags(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                              uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S,
                              const DeviceInfo& dev, cudaStream_t stream) {
    const size_t gsz = G32 ? 4 : 2;
    // one launch per run of indices that share (index >> 33); a single launch unless the buffer
    // crosses a multiple of 2^33 in global index space
    uint64_t done = 0;
    while (done < n) {
        const uint64_t idx = elem_offset + done;
        const uint64_t to_boundary = (static_cast<uint64_t>(1) << 33) - (idx & ((static_cast<uint64_t>(1) << 33) - 1));
        const uint64_t len = n - done < to_boundary ? n - done : to_boundary;
        uint16_t* ps = p + done;
        const void* gs = static_cast<const char*>(g) + done * gsz;
        uint16_t* ms = m + done;
        uint16_t* vs = v + done;
        const bool vec = aligned16(ps) && aligned16(gs) && aligned16(ms) && aligned16(vs);
        cudaError_t e;
        if (!vec)
            e = launch_flat_mode<G32, FLAGS, 0>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if ((idx & 7u) != 0 || !fast_path_allowed(S))
            e = launch_flat_mode<G32, FLAGS, 1>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if (needs_scale(S))
            e = launch_flat_mode<G32, FLAGS, 3>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else
            e = launch_flat_mode<G32, FLAGS, 2>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        if (e != cudaSuccess) return e;
        done += len;
    }
    return cudaSuccess;
}

template <bool G32>
cudaError_t launch_adamw_flat_g(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                                uint32_t tensor_id, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                                const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
#define SR_FLAT(F) launch_flat_flags<G32, F>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S, dev, stream)
    SR_DISPATCH_FLAGS(SR_FLAT)
#undef SR_FLAT
}

}  // namespace sradamw
