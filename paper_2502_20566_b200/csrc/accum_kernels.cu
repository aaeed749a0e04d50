// BF16 accumulator with stochastic rounding: acc <- Q_SR(acc + scale * g) (Eq. 2; Section 3 keeps every
// tensor in BF16, the accumulated gradient included) or the nearest-rounded Q of Eq. 1.
// FP32 arithmetic in registers, one rounding for the product and one for the sum.  Noise: rounding
// slot 3 of the group of eight elements (counter number 4 * (index >> 3) + 3), the one the optimizer
// step leaves unused.  6 bytes per element with BF16 terms (2 + 2 read, 2 written), 8 with FP32 terms.

#include "adamw_body.cuh"

namespace sradamw {

namespace {

constexpr uint32_t kAccumSlot = 3;

template <bool G32>
__device__ __forceinline__ float term_of(const void* g, uint64_t i) {
    return G32 ? static_cast<const float*>(g)[i]
               : __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(g)[i]) << 16);
}

__device__ __forceinline__ float accumulate(float acc, float g, float scale) {
    return __fadd_rn(acc, __fmul_rn(scale, g));
}

// one vector of eight: sums in FP32, rounded with the noise words w
template <bool SR>
__device__ __forceinline__ uint4 accumulate_vec(const uint4 av, const float (&ge)[8], const uint4 w, float scale) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t aw = word_of(av, j);
        const float s0 = accumulate(bf16_lo(aw), ge[2 * j], scale);
        const float s1 = accumulate(bf16_hi(aw), ge[2 * j + 1], scale);
        o[j] = pack_top_halves(round_sum_word_nan_safe<SR, false>(s0, word_of(w, j)),
                               round_sum_word_nan_safe<SR, true>(s1, word_of(w, j)));
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// MODE 0: element-wise; 1: 16-byte vectors straddling two noise groups (offset not a multiple of 8); 2: vectors, grouped
#ifndef SR_ACCUM_STRADDLE_MIN_BLOCKS
#define SR_ACCUM_STRADDLE_MIN_BLOCKS 1
#endif
template <bool G32, bool SR, int MODE>
__global__ void __launch_bounds__(kBlockThreads, MODE == 1 ? SR_ACCUM_STRADDLE_MIN_BLOCKS : 1)
k_sr_accumulate(uint16_t* acc, const void* g, uint64_t n, float scale, uint64_t elem_offset, uint32_t tensor_id,
                uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (MODE != 0) {
        // MODE 1 (every vector straddles two noise groups): every lane computes the call of the group its vector ends
        // in and takes the other group's words from the lane below (RowChain), whole rows of 32 vectors only (the
        // rest goes element by element); MODE 2: one thread, one vector, one call
        using Chain = RowChain<1u << kAccumSlot, false>;
        __shared__ uint4 heads[MODE == 1 ? (kBlockThreads / 32) * Chain::kTableEntries : 1];
        const uint64_t nvec = MODE == 1 ? (n >> 3) & ~static_cast<uint64_t>(31) : n >> 3;
        const uint32_t lane = threadIdx.x & 31u;
        const Chain chain{heads + (MODE == 1 ? (threadIdx.x >> 5) * Chain::kTableEntries : 0), elem_offset >> 3, stride,
                          static_cast<uint32_t>(elem_offset) & 7u, lane, 0u, tensor_id, seed_hi};
        uint32_t k = 0;
        uint64_t vec = tid;
        if (MODE == 2) {
            // two vectors per iteration: four 16-byte loads in flight per thread (838M elements: 0.812 -> 0.801 ms)
            for (; vec + stride < nvec; vec += 2 * stride) {
                const uint4 av0 = ld16(acc, vec), av1 = ld16(acc, vec + stride);
                float ge0[8], ge1[8];
                load_grad8<G32>(g, vec, ge0);
                load_grad8<G32>(g, vec + stride, ge1);
                uint4 w0 = make_uint4(0, 0, 0, 0), w1 = w0;
                if (SR) {
                    const uint64_t n0 = (((elem_offset >> 3) + vec) << 2) | kAccumSlot, n1 = n0 + (stride << 2);
                    w0 = philox4x32_10(static_cast<uint32_t>(n0), static_cast<uint32_t>(n0 >> 32), tensor_id, seed_hi, K);
                    w1 = philox4x32_10(static_cast<uint32_t>(n1), static_cast<uint32_t>(n1 >> 32), tensor_id, seed_hi, K);
                }
                st16(acc, vec, accumulate_vec<SR>(av0, ge0, w0, scale));
                st16(acc, vec + stride, accumulate_vec<SR>(av1, ge1, w1, scale));
            }
        }
        for (; vec < nvec; vec += stride, ++k) {
            const uint4 av = ld16(acc, vec);
            float ge[8];
            load_grad8<G32>(g, vec, ge);
            uint4 w = make_uint4(0, 0, 0, 0);
            if (SR && MODE == 1) {
                if ((k & 31u) == 0u) chain.refill(vec - lane, K);
                uint4 w4[4];
                chain.words(vec, k, K, w4);
                w = w4[kAccumSlot];
            } else if (SR) {
                const uint64_t number = (((elem_offset >> 3) + vec) << 2) | kAccumSlot;
                w = philox4x32_10(static_cast<uint32_t>(number), static_cast<uint32_t>(number >> 32), tensor_id, seed_hi, K);
            }
            st16(acc, vec, accumulate_vec<SR>(av, ge, w, scale));
        }
        done = nvec << 3;
    }
    for (uint64_t i = done + tid; i < n; i += stride) {
        const float s = accumulate(__uint_as_float(static_cast<uint32_t>(acc[i]) << 16), term_of<G32>(g, i), scale);
        const uint32_t r = SR ? noise_of_element(elem_offset + i, kAccumSlot, tensor_id, seed_hi, K) : 0u;
        acc[i] = static_cast<uint16_t>(round_sum_r16_nan_safe<SR>(s, r) >> 16);
    }
}

template <bool G32, bool SR, int MODE>
cudaError_t launch_accum_mode(uint16_t* acc, const void* g, uint64_t n, float scale, uint64_t elem_offset,
                              uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev,
                              cudaStream_t stream) {
    auto k = k_sr_accumulate<G32, SR, MODE>;
    const uint64_t items = MODE == 0 ? n : (n >> 3) + 8;
    k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(acc, g, n, scale, elem_offset, tensor_id, seed_hi, K);
    return cudaGetLastError();
}

template <bool G32, bool SR>
cudaError_t launch_accum_t(uint16_t* acc, const void* g, uint64_t n, float scale, uint64_t elem_offset, uint32_t tensor_id,
                           uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    if (!(aligned16(acc) && aligned16(g)))
        return launch_accum_mode<G32, SR, 0>(acc, g, n, scale, elem_offset, tensor_id, seed_hi, K, dev, stream);
    if (SR && (elem_offset & 7u) != 0)
        return launch_accum_mode<G32, SR, 1>(acc, g, n, scale, elem_offset, tensor_id, seed_hi, K, dev, stream);
    return launch_accum_mode<G32, SR, 2>(acc, g, n, scale, elem_offset, tensor_id, seed_hi, K, dev, stream);
}

}  // namespace

cudaError_t launch_accumulate(uint16_t* acc, const void* g, bool g_f32, uint64_t n, float scale, bool stochastic,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K,
                              const DeviceInfo& dev, cudaStream_t stream) {
#define SR_ACC(G, S) launch_accum_t<G, S>(acc, g, n, scale, elem_offset, tensor_id, seed_hi, K, dev, stream)
    if (g_f32) return stochastic ? SR_ACC(true, true) : SR_ACC(true, false);
    return stochastic ? SR_ACC(false, true) : SR_ACC(false, false);
#undef SR_ACC
}

}  // namespace sradamw
