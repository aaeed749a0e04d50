// Fused SR-AdamW kernels for sm_100a: one read of x, g, m, v and one write of x, m, v per element,
// with Philox, the FP32 update of Algorithm 1 and the dithering add all in registers.
//
// Memory-bound by design: 14 bytes per element with BF16 gradients, 16 with FP32 gradients.
// Each thread moves 8 consecutive elements per iteration with 16-byte loads and stores, a warp
// therefore touches 512 contiguous bytes per array; loads and stores carry the streaming
// (evict-first) hint because every byte is used exactly once.

#include "launch.h"

namespace sradamw {

namespace {

// ---- 16-byte streaming accesses ------------------------------------------------------------
__device__ __forceinline__ uint4 ld16(const void* base, uint64_t vec) {
    return __ldcs(reinterpret_cast<const uint4*>(base) + vec);
}
__device__ __forceinline__ void st16(void* base, uint64_t vec, uint4 val) {
    __stcs(reinterpret_cast<uint4*>(base) + vec, val);
}

// One pair of elements (the two halves of one 32-bit word of each BF16 array) whose first global
// index is idx0 + e.  PAIRED = true needs idx0 + e even (then both share one Philox call and, idx0
// being a multiple of 8, the pair counter low word cannot wrap inside a vector); PAIRED = false
// draws each element's noise on its own and is valid for any index.
template <uint32_t FLAGS, bool PAIRED>
__device__ __forceinline__ void step_pair(uint32_t pw, float g_even, float g_odd, uint32_t mw, uint32_t vw,
                                          uint64_t idx0, uint32_t e, uint32_t c2, uint32_t c3, float gscale,
                                          const PhiloxKeys& K, const StepScalars& S, uint32_t& po, uint32_t& mo,
                                          uint32_t& vo) {
    const ElementOut r0 = adamw_element(bf16_lo(pw), g_even, bf16_lo(mw), bf16_lo(vw), gscale, S);
    const ElementOut r1 = adamw_element(bf16_hi(pw), g_odd, bf16_hi(mw), bf16_hi(vw), gscale, S);
    uint32_t a0 = 0, a1 = 0, a2 = 0, b0 = 0, b1 = 0, b2 = 0;
    if (FLAGS != 0) {
        if (PAIRED) {
            uint32_t w0, w1, w2;
            philox4x32_10(static_cast<uint32_t>(idx0 >> 1) + (e >> 1), static_cast<uint32_t>(idx0 >> 33), c2, c3, K,
                          w0, w1, w2);
            a0 = noise_even(w0); a1 = noise_even(w1); a2 = noise_even(w2);
            b0 = noise_odd(w0); b1 = noise_odd(w1); b2 = noise_odd(w2);
        } else {
            noise_of_element(idx0 + e, c2, c3, K, a0, a1, a2);
            noise_of_element(idx0 + e + 1, c2, c3, K, b0, b1, b2);
        }
    }
    uint32_t sp0, sm0, sv0, sp1, sm1, sv1;
    round_element<FLAGS>(r0, a0, a1, a2, sp0, sm0, sv0);
    round_element<FLAGS>(r1, b0, b1, b2, sp1, sm1, sv1);
    po = pack_top_halves(sp0, sp1);
    mo = pack_top_halves(sm0, sm1);
    vo = pack_top_halves(sv0, sv1);
}

// Eight consecutive elements starting at global index idx0; element arrays addressed by `vec`.
template <bool G32, uint32_t FLAGS, bool PAIRED>
__device__ __forceinline__ void step_vec8(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t vec,
                                          uint64_t idx0, uint32_t c2, uint32_t c3, float gscale, const PhiloxKeys& K,
                                          const StepScalars& S) {
    const uint4 pv = ld16(p, vec);
    const uint4 mv = ld16(m, vec);
    const uint4 vv = ld16(v, vec);
    float ge[8];
    if (G32) {
        const uint4 g0 = ld16(g, 2 * vec);
        const uint4 g1 = ld16(g, 2 * vec + 1);
        ge[0] = __uint_as_float(g0.x); ge[1] = __uint_as_float(g0.y);
        ge[2] = __uint_as_float(g0.z); ge[3] = __uint_as_float(g0.w);
        ge[4] = __uint_as_float(g1.x); ge[5] = __uint_as_float(g1.y);
        ge[6] = __uint_as_float(g1.z); ge[7] = __uint_as_float(g1.w);
    } else {
        const uint4 gv = ld16(g, vec);
        ge[0] = bf16_lo(gv.x); ge[1] = bf16_hi(gv.x);
        ge[2] = bf16_lo(gv.y); ge[3] = bf16_hi(gv.y);
        ge[4] = bf16_lo(gv.z); ge[5] = bf16_hi(gv.z);
        ge[6] = bf16_lo(gv.w); ge[7] = bf16_hi(gv.w);
    }
    uint4 po, mo, vo;
    step_pair<FLAGS, PAIRED>(pv.x, ge[0], ge[1], mv.x, vv.x, idx0, 0, c2, c3, gscale, K, S, po.x, mo.x, vo.x);
    step_pair<FLAGS, PAIRED>(pv.y, ge[2], ge[3], mv.y, vv.y, idx0, 2, c2, c3, gscale, K, S, po.y, mo.y, vo.y);
    step_pair<FLAGS, PAIRED>(pv.z, ge[4], ge[5], mv.z, vv.z, idx0, 4, c2, c3, gscale, K, S, po.z, mo.z, vo.z);
    step_pair<FLAGS, PAIRED>(pv.w, ge[6], ge[7], mv.w, vv.w, idx0, 6, c2, c3, gscale, K, S, po.w, mo.w, vo.w);
    st16(p, vec, po);
    st16(m, vec, mo);
    st16(v, vec, vo);
}

// One element with 2-byte accesses: ragged tails and buffers that are not 16-byte aligned.
template <bool G32, uint32_t FLAGS>
__device__ __forceinline__ void step_scalar(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t i,
                                            uint64_t idx, uint32_t c2, uint32_t c3, float gscale, const PhiloxKeys& K,
                                            const StepScalars& S) {
    const float x = __uint_as_float(static_cast<uint32_t>(p[i]) << 16);
    const float mi = __uint_as_float(static_cast<uint32_t>(m[i]) << 16);
    const float vi = __uint_as_float(static_cast<uint32_t>(v[i]) << 16);
    const float gi = G32 ? static_cast<const float*>(g)[i]
                         : __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(g)[i]) << 16);
    const ElementOut r = adamw_element(x, gi, mi, vi, gscale, S);
    uint32_t w0 = 0, w1 = 0, w2 = 0;
    if (FLAGS != 0) noise_of_element(idx, c2, c3, K, w0, w1, w2);
    uint32_t sp, sm, sv;
    round_element<FLAGS>(r, w0, w1, w2, sp, sm, sv);
    p[i] = static_cast<uint16_t>(sp >> 16);
    m[i] = static_cast<uint16_t>(sm >> 16);
    v[i] = static_cast<uint16_t>(sv >> 16);
}

// ---- flat buffer ---------------------------------------------------------------------------
// Persistent grid: thread t of the grid takes vectors t, t + T, t + 2T, ... (T = threads in the
// grid).  VEC = false is the element-wise kernel for unaligned buffers.
template <bool G32, uint32_t FLAGS, bool PAIRED, bool VEC>
__global__ void __launch_bounds__(kBlockThreads)
k_sr_adamw_flat(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K,
                const __grid_constant__ StepScalars S) {
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    if (VEC) {
        const uint64_t nvec = n >> 3;
        for (uint64_t vec = tid; vec < nvec; vec += stride)
            step_vec8<G32, FLAGS, PAIRED>(p, g, m, v, vec, elem_offset + (vec << 3), tensor_id, seed_hi, gscale, K, S);
        const uint64_t done = nvec << 3;
        if (tid < n - done)
            step_scalar<G32, FLAGS>(p, g, m, v, done + tid, elem_offset + done + tid, tensor_id, seed_hi, gscale, K, S);
    } else {
        for (uint64_t i = tid; i < n; i += stride)
            step_scalar<G32, FLAGS>(p, g, m, v, i, elem_offset + i, tensor_id, seed_hi, gscale, K, S);
    }
}

// ---- tensor list ---------------------------------------------------------------------------
// Blocks walk the chunk table; a chunk is up to kMtChunkElems consecutive elements of one tensor.
// Element indices restart at 0 in every tensor and chunk starts are multiples of 8, so vectors
// always hold aligned pairs.
template <bool G32, uint32_t FLAGS>
__global__ void __launch_bounds__(kBlockThreads)
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
            for (uint32_t j = threadIdx.x; j < nvec; j += blockDim.x)
                step_vec8<G32, FLAGS, true>(T.p, T.g, T.m, T.v, vec0 + j, start + (static_cast<uint64_t>(j) << 3), c2,
                                             seed_hi, gscale, K, S);
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

// ---- standalone Q_SR cast ------------------------------------------------------------------
// Uses the x slot (word 0) of the same noise layout: one Philox call per two elements.
template <bool PAIRED>
__device__ __forceinline__ uint32_t downcast_pair(uint32_t b_even, uint32_t b_odd, uint64_t idx0, uint32_t e,
                                                  uint32_t c2, uint32_t c3, const PhiloxKeys& K) {
    uint32_t r_even, r_odd, w1, w2;
    if (PAIRED) {
        uint32_t w0;
        philox4x32_10(static_cast<uint32_t>(idx0 >> 1) + (e >> 1), static_cast<uint32_t>(idx0 >> 33), c2, c3, K, w0, w1, w2);
        r_even = noise_even(w0);
        r_odd = noise_odd(w0);
    } else {
        noise_of_element(idx0 + e, c2, c3, K, r_even, w1, w2);
        noise_of_element(idx0 + e + 1, c2, c3, K, r_odd, w1, w2);
    }
    const uint32_t s0 = is_nan_bits(b_even) ? (kQuietNaNbf16 << 16) : sr_sum(b_even, r_even);
    const uint32_t s1 = is_nan_bits(b_odd) ? (kQuietNaNbf16 << 16) : sr_sum(b_odd, r_odd);
    return pack_top_halves(s0, s1);
}

template <bool PAIRED, bool VEC>
__global__ void __launch_bounds__(kBlockThreads)
k_sr_downcast(const float* __restrict__ src, uint16_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
              uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (VEC) {
        const uint64_t nvec = n >> 3;
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            const uint4 a = ld16(src, 2 * vec);
            const uint4 b = ld16(src, 2 * vec + 1);
            const uint64_t idx0 = elem_offset + (vec << 3);
            uint4 o;
            o.x = downcast_pair<PAIRED>(a.x, a.y, idx0, 0, tensor_id, seed_hi, K);
            o.y = downcast_pair<PAIRED>(a.z, a.w, idx0, 2, tensor_id, seed_hi, K);
            o.z = downcast_pair<PAIRED>(b.x, b.y, idx0, 4, tensor_id, seed_hi, K);
            o.w = downcast_pair<PAIRED>(b.z, b.w, idx0, 6, tensor_id, seed_hi, K);
            st16(dst, vec, o);
        }
        done = nvec << 3;
    }
    for (uint64_t i = done + tid; i < n; i += stride) {
        uint32_t r0, r1, r2;
        noise_of_element(elem_offset + i, tensor_id, seed_hi, K, r0, r1, r2);
        const uint32_t b = __float_as_uint(src[i]);
        dst[i] = static_cast<uint16_t>((is_nan_bits(b) ? (kQuietNaNbf16 << 16) : sr_sum(b, r0)) >> 16);
    }
}

// ---- launch helpers ------------------------------------------------------------------------
inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

template <typename Kernel>
int resident_blocks(Kernel kernel, const DeviceInfo& dev) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kBlockThreads, 0) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    return per_sm * dev.sm_count;
}

// grid for `work_items` thread-items: no more blocks than are resident at once, no more than needed
template <typename Kernel>
unsigned grid_for(Kernel kernel, uint64_t work_items, const DeviceInfo& dev) {
    const uint64_t needed = (work_items + kBlockThreads - 1) / kBlockThreads;
    const uint64_t resident = static_cast<uint64_t>(resident_blocks(kernel, dev));
    const uint64_t g = needed < resident ? needed : resident;
    return static_cast<unsigned>(g < 1 ? 1 : g);
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_flat_t(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                          uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S,
                          const DeviceInfo& dev, cudaStream_t stream) {
    const bool vec = aligned16(p) && aligned16(g) && aligned16(m) && aligned16(v);
    const uint64_t vec_items = (n >> 3) + 8;   // the extra 8 keep enough threads for the ragged tail
    if (!vec) {
        auto k = k_sr_adamw_flat<G32, FLAGS, false, false>;
        k<<<grid_for(k, n, dev), kBlockThreads, 0, stream>>>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S);
    } else if ((elem_offset & 7u) == 0) {
        auto k = k_sr_adamw_flat<G32, FLAGS, true, true>;
        k<<<grid_for(k, vec_items, dev), kBlockThreads, 0, stream>>>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S);
    } else {
        auto k = k_sr_adamw_flat<G32, FLAGS, false, true>;
        k<<<grid_for(k, vec_items, dev), kBlockThreads, 0, stream>>>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S);
    }
    return cudaGetLastError();
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_mt_t(const MtTensor* tensors, const MtChunk* chunks, uint32_t num_chunks, uint32_t tensor_id_base,
                        uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev,
                        cudaStream_t stream) {
    auto k = k_sr_adamw_mt<G32, FLAGS>;
    const unsigned resident = static_cast<unsigned>(resident_blocks(k, dev));
    const unsigned grid = num_chunks < resident ? num_chunks : resident;
    k<<<grid, kBlockThreads, 0, stream>>>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S);
    return cudaGetLastError();
}

}  // namespace

#define SR_DISPATCH_FLAGS(G32, CALL)                  \
    switch (flags & 7u) {                             \
        case 0: return CALL(G32, 0);                  \
        case 1: return CALL(G32, 1);                  \
        case 2: return CALL(G32, 2);                  \
        case 3: return CALL(G32, 3);                  \
        case 4: return CALL(G32, 4);                  \
        case 5: return CALL(G32, 5);                  \
        case 6: return CALL(G32, 6);                  \
        default: return CALL(G32, 7);                 \
    }

cudaError_t launch_adamw_flat(uint16_t* p, const void* g, bool g_f32, uint16_t* m, uint16_t* v, uint64_t n,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, uint32_t flags,
                              const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
#define SR_FLAT(G32, F) launch_flat_t<G32, F>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S, dev, stream)
    if (g_f32) {
        SR_DISPATCH_FLAGS(true, SR_FLAT)
    } else {
        SR_DISPATCH_FLAGS(false, SR_FLAT)
    }
#undef SR_FLAT
}

cudaError_t launch_adamw_mt(const MtTensor* tensors, const MtChunk* chunks, uint32_t num_chunks, bool g_f32,
                            uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
#define SR_MT(G32, F) launch_mt_t<G32, F>(tensors, chunks, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream)
    if (g_f32) {
        SR_DISPATCH_FLAGS(true, SR_MT)
    } else {
        SR_DISPATCH_FLAGS(false, SR_MT)
    }
#undef SR_MT
}

cudaError_t launch_downcast(const float* src, uint16_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                            uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    const bool vec = aligned16(src) && aligned16(dst);
    if (!vec) {
        auto k = k_sr_downcast<false, false>;
        k<<<grid_for(k, n, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    } else if ((elem_offset & 7u) == 0) {
        auto k = k_sr_downcast<true, true>;
        k<<<grid_for(k, (n >> 3) + 8, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    } else {
        auto k = k_sr_downcast<false, true>;
        k<<<grid_for(k, (n >> 3) + 8, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    }
    return cudaGetLastError();
}

}  // namespace sradamw
