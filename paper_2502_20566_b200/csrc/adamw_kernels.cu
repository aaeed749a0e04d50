// Entry points of the kernel layer for the fused step (dispatch on the gradient type) and the
// standalone stochastic-rounding cast.
#include "adamw_body.cuh"

namespace sradamw {

cudaError_t launch_adamw_flat(uint16_t* p, const void* g, bool g_f32, uint16_t* m, uint16_t* v, uint64_t n,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, uint32_t flags,
                              const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    return g_f32 ? launch_adamw_flat_g<true>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, flags, K, S, dev, stream)
                 : launch_adamw_flat_g<false>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, flags, K, S, dev, stream);
}

cudaError_t launch_adamw_mt(const MtWork* work, uint32_t num_chunks, bool g_f32,
                            uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    return g_f32 ? launch_adamw_mt_g<true>(work, num_chunks, tensor_id_base, seed_hi, flags, K, S, dev, stream)
                 : launch_adamw_mt_g<false>(work, num_chunks, tensor_id_base, seed_hi, flags, K, S, dev, stream);
}

// ---- standalone Q_SR cast ------------------------------------------------------------------
// Slot 0 of the noise layout: ONE Philox call per eight elements.  6 bytes per element.
namespace {

__device__ __forceinline__ uint32_t cast_pair(uint32_t b_even, uint32_t b_odd, uint32_t word) {
    const uint32_t s0 = is_nan_bits(b_even) ? (kQuietNaNbf16 << 16) : sr_sum_lo(b_even, word);
    const uint32_t s1 = is_nan_bits(b_odd) ? (kQuietNaNbf16 << 16) : sr_sum_hi(b_odd, word);
    return pack_top_halves(s0, s1);
}

// MODE 0: element-wise; 1: vectors straddling two noise groups (offset not a multiple of 8); 2: vectors, grouped
template <int MODE>
__global__ void __launch_bounds__(kBlockThreads)
k_sr_downcast(const float* __restrict__ src, uint16_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
              uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (MODE == 1) {
        // every vector straddles two noise groups: every lane computes the call of the group its vector ends in and
        // takes the other group's words from the lane below (RowChain)
        using Chain = RowChain<1u, false>;
        __shared__ uint4 heads[(kBlockThreads / 32) * Chain::kTableEntries];
        const uint64_t row_vecs = (n >> 3) & ~static_cast<uint64_t>(31);   // whole rows of 32 vectors; the rest goes element by element
        const uint32_t lane = threadIdx.x & 31u;
        const Chain chain{heads + (threadIdx.x >> 5) * Chain::kTableEntries, elem_offset >> 3, stride,
                          static_cast<uint32_t>(elem_offset) & 7u, lane, 0u, tensor_id, seed_hi};
        uint32_t k = 0;
        for (uint64_t vec = tid; vec < row_vecs; vec += stride, ++k) {
            const uint4 a = ld16(src, 2 * vec);
            const uint4 b = ld16(src, 2 * vec + 1);
            if ((k & 31u) == 0u) chain.refill(vec - lane, K);
            uint4 w4[4];
            chain.words(vec, k, K, w4);
            const uint4 w = w4[0];
            uint4 o;
            o.x = cast_pair(a.x, a.y, w.x);
            o.y = cast_pair(a.z, a.w, w.y);
            o.z = cast_pair(b.x, b.y, w.z);
            o.w = cast_pair(b.z, b.w, w.w);
            st16(dst, vec, o);
        }
        done = row_vecs << 3;
    } else if (MODE == 2) {
        const uint64_t nvec = n >> 3;
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            const uint4 a = ld16(src, 2 * vec);
            const uint4 b = ld16(src, 2 * vec + 1);
            const uint64_t idx0 = elem_offset + (vec << 3);
            const uint4 w = philox4x32_10(static_cast<uint32_t>(idx0 >> 1), static_cast<uint32_t>(idx0 >> 33), tensor_id, seed_hi, K);
            uint4 o;
            o.x = cast_pair(a.x, a.y, w.x);
            o.y = cast_pair(a.z, a.w, w.y);
            o.z = cast_pair(b.x, b.y, w.z);
            o.w = cast_pair(b.z, b.w, w.w);
            st16(dst, vec, o);
        }
        done = nvec << 3;
    }
    for (uint64_t i = done + tid; i < n; i += stride) {
        const uint32_t r = noise_of_element(elem_offset + i, 0, tensor_id, seed_hi, K);
        dst[i] = static_cast<uint16_t>(round_sum_r16_nan_safe<true>(src[i], r) >> 16);
    }
}

template <int MODE>
cudaError_t launch_cast_mode(const float* src, uint16_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                             uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    auto k = k_sr_downcast<MODE>;
    const uint64_t items = MODE == 0 ? n : (n >> 3) + 8;
    k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_downcast(const float* src, uint16_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                            uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    if (!(aligned16(src) && aligned16(dst)))
        return launch_cast_mode<0>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream);
    if ((elem_offset & 7u) != 0)
        return launch_cast_mode<1>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream);
    return launch_cast_mode<2>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream);
}

}  // namespace sradamw
