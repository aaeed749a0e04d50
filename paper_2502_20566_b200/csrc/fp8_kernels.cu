// Stochastic-rounding casts FP32 -> FP8 (E4M3 / E5M2) and FP32 -> FP4 (E2M1): Eq. 2 on the 8-bit and
// 4-bit grids, the extension the paper's conclusion names.  5 bytes per element (4 read, 1 written)
// for FP8, 4.5 for FP4 (two codes per byte).  32 noise bits per element, one Philox call per four
// consecutive elements (counter number = index >> 2, word = index & 3).

#include "adamw_body.cuh"

namespace sradamw {

namespace {

// FMT 0: E4M3, 1: E5M2, 2: E2M1
constexpr int kE4M3 = 0, kE5M2 = 1, kE2M1 = 2;

template <int FMT>
struct Small {
    static constexpr int M = FMT == kE5M2 ? 2 : FMT == kE4M3 ? 3 : 1;
    static constexpr int kBias = FMT == kE5M2 ? 15 : FMT == kE4M3 ? 7 : 1;
    static constexpr uint32_t kMaxCode = FMT == kE5M2 ? 0x7Bu : FMT == kE4M3 ? 0x7Eu : 0x7u;   // 57344, 448, 6
    static constexpr uint32_t kMaxBits = FMT == kE5M2 ? 0x47600000u : FMT == kE4M3 ? 0x43E00000u : 0x40C00000u;   // as FP32
    static constexpr uint32_t kInfCode = 0x7Cu;                              // E5M2 only: the others have no infinity
    static constexpr uint32_t kMinBiasedExp = 127 + 1 - kBias;               // FP32 exponent field of the smallest normal level
};

// The magnitude code of one value (sign handled by the caller).  a = |x| lies in the binade
// Eq = max(E, 1 - bias); y = a / 2^(Eq - M) = k + f; move to level k + 1 iff r < floor(f * 2^32).
// Evaluated with exact FP32 operations, which keeps most of the work off the integer pipe that
// bounds this kernel: y = a * 2^(M - Eq) is a scaling by a power of two (exact, subnormal a
// included; y < 2^(M+1)); adding 2^23 with rounding toward zero leaves k in the low bits of the sum;
// f = y - k is exact; f * 2^32 < 2^32 is exact and its truncation to an integer is the threshold.
// The code of level k' is ((Eq + bias - 1) << M) + k' for subnormal and normal levels alike.
// Magnitudes at or beyond the largest level (infinity and NaN included, whose y is meaningless)
// are replaced at the end.
template <int FMT>
__device__ __forceinline__ uint32_t sr_fp8_magnitude(uint32_t abits, uint32_t r) {
    using F = Small<FMT>;
    const uint32_t e = abits >> 23;                                            // biased FP32 exponent
    const uint32_t eqb = e < F::kMinBiasedExp ? F::kMinBiasedExp : e;          // Eq + 127
    const float scale = __uint_as_float(((254u + F::M) << 23) - (eqb << 23));  // 2^(M - Eq)
    const float y = __fmul_rn(__uint_as_float(abits), scale);
    const float t = __fadd_rz(y, 8388608.0f);                                  // 2^23 + k
    const float f = __fsub_rn(y, __fsub_rn(t, 8388608.0f));
    const uint32_t threshold = __float2uint_rz(__fmul_rn(f, 4294967296.0f));
    uint32_t code = (eqb << F::M) + __float_as_uint(t) - (0x4B000000u + (F::kMinBiasedExp << F::M)) + (r < threshold ? 1u : 0u);
    code = abits >= F::kMaxBits ? F::kMaxCode : code;
    if (FMT == kE2M1) return code;
    if (FMT == kE5M2) code = abits == 0x7F800000u ? F::kInfCode : code;
    return abits > 0x7F800000u ? 0x7Fu : code;                                 // NaN -> 0x7F (its sign is dropped below)
}

// The same for two values at once with the packed FP32 instructions of sm_100 (each lane is the scalar
// operation, rounding mode included): half the floating-point instructions.
__device__ __forceinline__ uint64_t add_rz2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

template <int FMT>
__device__ __forceinline__ uint32_t finish_code(uint32_t abits, uint32_t eqb, float t, float fscaled, uint32_t r) {
    using F = Small<FMT>;
    const uint32_t threshold = __float2uint_rz(fscaled);
    uint32_t code = (eqb << F::M) + __float_as_uint(t) - (0x4B000000u + (F::kMinBiasedExp << F::M)) + (r < threshold ? 1u : 0u);
    code = abits >= F::kMaxBits ? F::kMaxCode : code;
    if (FMT == kE2M1) return code;
    if (FMT == kE5M2) code = abits == 0x7F800000u ? F::kInfCode : code;
    return abits > 0x7F800000u ? 0x7Fu : code;
}

template <int FMT>
__device__ __forceinline__ void sr_fp8_magnitude2(uint32_t a0, uint32_t a1, uint32_t r0, uint32_t r1, uint32_t& c0, uint32_t& c1) {
    using F = Small<FMT>;
    const uint32_t e0 = a0 >> 23, e1 = a1 >> 23;
    const uint32_t q0 = e0 < F::kMinBiasedExp ? F::kMinBiasedExp : e0, q1 = e1 < F::kMinBiasedExp ? F::kMinBiasedExp : e1;
    const float s0 = __uint_as_float(((254u + F::M) << 23) - (q0 << 23)), s1 = __uint_as_float(((254u + F::M) << 23) - (q1 << 23));
    const uint64_t y = mul2(pack2(__uint_as_float(a0), __uint_as_float(a1)), pack2(s0, s1));
    const uint64_t magic = dup2(8388608.0f);
    const uint64_t t = add_rz2(y, magic);
    const uint64_t f = sub2(y, sub2(t, magic));
    const uint64_t fs = mul2(f, dup2(4294967296.0f));
    float t0, t1, f0, f1;
    unpack2(t, t0, t1);
    unpack2(fs, f0, f1);
    c0 = finish_code<FMT>(a0, q0, t0, f0, r0);
    c1 = finish_code<FMT>(a1, q1, t1, f1, r1);
}

template <int FMT>
__device__ __forceinline__ uint32_t sr_fp8_code(uint32_t fbits, uint32_t r) {
    const uint32_t abits = fbits & 0x7FFFFFFFu;
    const uint32_t sign = abits > 0x7F800000u ? 0u : ((fbits >> 24) & 0x80u);
    return sign | sr_fp8_magnitude<FMT>(abits, r);
}

// E2M1: sign in bit 3 (kept for NaN too), magnitude code in bits 0..2
__device__ __forceinline__ uint32_t sr_fp4_code(uint32_t fbits, uint32_t r) {
    return ((fbits >> 28) & 0x8u) | sr_fp8_magnitude<kE2M1>(fbits & 0x7FFFFFFFu, r);
}

// four values -> four 4-bit codes in bits 0..15 (element j in bits 4j..4j+3)
__device__ __forceinline__ uint32_t cast4_fp4(const uint4 x, const uint4 w) {
    uint32_t n0, n1, n2, n3;
    sr_fp8_magnitude2<kE2M1>(x.x & 0x7FFFFFFFu, x.y & 0x7FFFFFFFu, w.x, w.y, n0, n1);
    sr_fp8_magnitude2<kE2M1>(x.z & 0x7FFFFFFFu, x.w & 0x7FFFFFFFu, w.z, w.w, n2, n3);
    n0 |= (x.x >> 28) & 0x8u;
    n1 |= (x.y >> 28) & 0x8u;
    n2 |= (x.z >> 28) & 0x8u;
    n3 |= (x.w >> 28) & 0x8u;
    return (n1 * 16u + n0) + (n3 * 16u + n2) * 256u;
}

__device__ __forceinline__ uint32_t noise32_of_element(uint64_t idx, uint32_t c2, uint32_t c3, const PhiloxKeys& K) {
    const uint64_t number = idx >> 2;
    const uint4 w = philox4x32_10(static_cast<uint32_t>(number), static_cast<uint32_t>(number >> 32), c2, c3, K);
    const uint32_t e = static_cast<uint32_t>(idx) & 3u;
    return e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w;
}

// four values -> four bytes; the four sign bits are gathered with two byte permutes
template <int FMT>
__device__ __forceinline__ uint32_t cast4(const uint4 x, const uint4 w) {
    const uint32_t ax = x.x & 0x7FFFFFFFu, ay = x.y & 0x7FFFFFFFu, az = x.z & 0x7FFFFFFFu, aw = x.w & 0x7FFFFFFFu;
    uint32_t m0, m1, m2, m3;
    sr_fp8_magnitude2<FMT>(ax, ay, w.x, w.y, m0, m1);
    sr_fp8_magnitude2<FMT>(az, aw, w.z, w.w, m2, m3);
    const uint32_t mags = __byte_perm(__byte_perm(m0, m1, 0x0040), __byte_perm(m2, m3, 0x0040), 0x5410);
    const uint32_t tops = __byte_perm(__byte_perm(x.x, x.y, 0x0073), __byte_perm(x.z, x.w, 0x0073), 0x5410);
    // a NaN code (0x7F) keeps no sign: mask the sign bit where the magnitude byte is 0x7F with all of bits 0..6 set
    const uint32_t is_nan = ((mags & 0x7F7F7F7Fu) + 0x01010101u) & 0x80808080u;
    return mags | (tops & 0x80808080u & ~is_nan);
}

// VEC: 16 elements per thread-iteration (4 x 16-byte loads, 1 x 16-byte store); needs both buffers
// 16-byte aligned and elem_offset a multiple of 4 (whole noise groups).
template <int FMT, bool VEC>
__global__ void __launch_bounds__(kBlockThreads)
k_sr_downcast_fp8(const float* __restrict__ src, uint8_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
                  uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (VEC) {
        const uint64_t nvec = n >> 4;
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            const uint4 a = ld16(src, 4 * vec), b = ld16(src, 4 * vec + 1), c = ld16(src, 4 * vec + 2), d = ld16(src, 4 * vec + 3);
            const uint64_t number = (elem_offset + (vec << 4)) >> 2;
            const uint32_t c0 = static_cast<uint32_t>(number), c1 = static_cast<uint32_t>(number >> 32);
            uint4 o;
            o.x = cast4<FMT>(a, philox4x32_10(c0, c1, tensor_id, seed_hi, K));
            o.y = cast4<FMT>(b, philox4x32_10(c0 + 1, c1, tensor_id, seed_hi, K));
            o.z = cast4<FMT>(c, philox4x32_10(c0 + 2, c1, tensor_id, seed_hi, K));
            o.w = cast4<FMT>(d, philox4x32_10(c0 + 3, c1, tensor_id, seed_hi, K));
            st16(dst, vec, o);
        }
        done = nvec << 4;
    }
    for (uint64_t i = done + tid; i < n; i += stride)
        dst[i] = static_cast<uint8_t>(sr_fp8_code<FMT>(__float_as_uint(src[i]), noise32_of_element(elem_offset + i, tensor_id, seed_hi, K)));
}

// E2M1, two codes per byte (element 2j in bits 0..3 of byte j).  VEC: 16 elements per
// thread-iteration (4 x 16-byte loads, one 8-byte store); needs src 16-byte and dst 8-byte aligned
// and elem_offset a multiple of 16.  The rest (and everything without VEC) goes byte by byte, one
// thread per output byte.
template <bool VEC>
__global__ void __launch_bounds__(kBlockThreads)
k_sr_downcast_fp4(const float* __restrict__ src, uint8_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
                  uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (VEC) {
        const uint64_t nvec = n >> 4;
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            const uint4 a = ld16(src, 4 * vec), b = ld16(src, 4 * vec + 1), c = ld16(src, 4 * vec + 2), d = ld16(src, 4 * vec + 3);
            const uint64_t number = (elem_offset + (vec << 4)) >> 2;
            const uint32_t c0 = static_cast<uint32_t>(number), c1 = static_cast<uint32_t>(number >> 32);
            const uint32_t lo = cast4_fp4(a, philox4x32_10(c0, c1, tensor_id, seed_hi, K)) |
                                (cast4_fp4(b, philox4x32_10(c0 + 1, c1, tensor_id, seed_hi, K)) << 16);
            const uint32_t hi = cast4_fp4(c, philox4x32_10(c0 + 2, c1, tensor_id, seed_hi, K)) |
                                (cast4_fp4(d, philox4x32_10(c0 + 3, c1, tensor_id, seed_hi, K)) << 16);
            __stcs(reinterpret_cast<uint2*>(dst) + vec, make_uint2(lo, hi));
        }
        done = nvec << 4;
    }
    const uint64_t nbytes = (n + 1) >> 1;
    for (uint64_t j = (done >> 1) + tid; j < nbytes; j += stride) {
        const uint64_t i0 = 2 * j, i1 = i0 + 1;
        uint32_t byte = sr_fp4_code(__float_as_uint(src[i0]), noise32_of_element(elem_offset + i0, tensor_id, seed_hi, K));
        if (i1 < n)
            byte |= sr_fp4_code(__float_as_uint(src[i1]), noise32_of_element(elem_offset + i1, tensor_id, seed_hi, K)) << 4;
        dst[j] = static_cast<uint8_t>(byte);
    }
}

template <int FMT, bool VEC>
cudaError_t launch_fp8_t(const float* src, uint8_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                         uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    auto k = k_sr_downcast_fp8<FMT, VEC>;
    const uint64_t items = VEC ? (n >> 4) + 16 : n;
    k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_downcast_fp8(const float* src, uint8_t* dst, uint64_t n, bool e5m2, uint64_t elem_offset,
                                uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev,
                                cudaStream_t stream) {
    // the low word of the group number must not wrap inside a 16-element vector: offset multiple of 16
    const bool vec = aligned16(src) && aligned16(dst) && (elem_offset & 15u) == 0;
    if (e5m2) return vec ? launch_fp8_t<kE5M2, true>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream)
                         : launch_fp8_t<kE5M2, false>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream);
    return vec ? launch_fp8_t<kE4M3, true>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream)
               : launch_fp8_t<kE4M3, false>(src, dst, n, elem_offset, tensor_id, seed_hi, K, dev, stream);
}

cudaError_t launch_downcast_fp4(const float* src, uint8_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                                uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    const bool vec = aligned16(src) && (reinterpret_cast<uintptr_t>(dst) & 7u) == 0 && (elem_offset & 15u) == 0;
    const uint64_t items = (vec ? (n >> 4) + 16 : (n + 1) >> 1);
    if (vec) {
        auto k = k_sr_downcast_fp4<true>;
        k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    } else {
        auto k = k_sr_downcast_fp4<false>;
        k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
    }
    return cudaGetLastError();
}

}  // namespace sradamw
