// Stochastic-rounding casts FP32 -> FP8 (E4M3 / E5M2) and FP32 -> FP4 (E2M1): Eq. 2 on the 8-bit and
// 4-bit grids, the extension the paper's conclusion names.  5 bytes per element (4 read, 1 written)
// for FP8, 4.5 for FP4 (two codes per byte).  32 noise bits per element, one Philox call per four
// consecutive elements (counter number = index >> 2, word = index & 3).

#include "adamw_body.cuh"

namespace sradamw {

namespace {

// FMT 0: E4M3, 1: E5M2, 2: E2M1
constexpr int kE4M3 = 0, kE5M2 = 1, kE2M1 = 2;

constexpr uint32_t kE5M2InfCode = 0x7Cu;   // the other two formats have no infinity

template <int FMT>
struct Small {
    static constexpr int M = FMT == kE5M2 ? 2 : FMT == kE4M3 ? 3 : 1;
    static constexpr int kBias = FMT == kE5M2 ? 15 : FMT == kE4M3 ? 7 : 1;
    // largest level as FP32: 57344 (code 0x7B), 448 (code 0x7E), 6 (code 0x7)
    static constexpr uint32_t kMaxBits = FMT == kE5M2 ? 0x47600000u : FMT == kE4M3 ? 0x43E00000u : 0x40C00000u;
    static constexpr uint32_t kMinBiasedExp = 127 + 1 - kBias;               // FP32 exponent field of the smallest normal level
};

// Multipliers read from constant memory.  The integer (ALU) pipe and the heavy half of the FMA pipe, which takes
// every integer multiply-add, bound these kernels about equally.  Where a subtraction or a shift-add is better
// placed on the FMA pipe it is written as a multiply-add whose multiplier is read from memory: a runtime value to
// the compiler, which would otherwise turn it back into an ALU instruction.  Which operation sits on which pipe
// was settled by measurement on B200 (2^28 values; see each use).
__constant__ uint32_t kMul[3] = {0xFFFFFFFFu, 256u, 65536u};
__device__ __forceinline__ uint32_t mul_minus1() { return kMul[0]; }
__device__ __forceinline__ uint32_t mul_256() { return kMul[1]; }
__device__ __forceinline__ uint32_t mul_65536() { return kMul[2]; }

// The magnitude code of one value (sign handled by the caller).  a = |x| lies in the binade
// Eq = max(E, 1 - bias); y = a / 2^(Eq - M) = k + f; move to level k + 1 iff r < floor(f * 2^32).
//   a  = min(|x|, largest level)      one float minimum: saturation and infinity land on the largest level with
//                                     f = 0, which never moves up
//   Eq from max(a, smallest normal level), exponent field only
//   z  = a * 2^(32 + M - Eq)          a scaling by a power of two: exact, subnormal a included; z < 2^(33 + M)
//   Z  = z truncated to a 64-bit integer = (k : floor(f * 2^32))
//   code = ((Eq + bias - 1) << M) + k + (r < low word of Z)      subnormal and normal levels alike
// NAN_ABOVE (the FP8 formats): minimum and maximum propagate a NaN, its exponent field is all ones and Z = 0, so
// its code comes out far above every level's and the caller's min(code, 0x7F) writes the NaN pattern.  Otherwise
// (E2M1, which has no NaN) a NaN lands on the largest level like infinity.
template <int FMT, bool NAN_ABOVE>
__device__ __forceinline__ uint32_t sr_small_magnitude(float x, uint32_t r) {
    using F = Small<FMT>;
    float a, an;
    if (NAN_ABOVE) {
        asm("min.NaN.f32 %0, %1, %2;" : "=f"(a) : "f"(fabsf(x)), "f"(__uint_as_float(F::kMaxBits)));
        asm("max.NaN.f32 %0, %1, %2;" : "=f"(an) : "f"(a), "f"(__uint_as_float(F::kMinBiasedExp << 23)));
    } else {
        a = fminf(fabsf(x), __uint_as_float(F::kMaxBits));
        an = fmaxf(a, __uint_as_float(F::kMinBiasedExp << 23));
    }
    const uint32_t eqbits = __float_as_uint(an) & 0x7F800000u;                            // (Eq + 127) << 23
    // 2^(32 + M - Eq): exponent field 127 + 32 + M - (Eq + 127) + 127, on the FMA pipe (0.354 -> 0.330 ms for E4M3)
    const float scale = __uint_as_float(eqbits * mul_minus1() + ((286u + F::M) << 23));
    const unsigned long long Z = __float2ull_rz(__fmul_rn(a, scale));
    constexpr uint32_t kBase = F::kMinBiasedExp << F::M;
    const uint32_t zlo = static_cast<uint32_t>(Z), zhi = static_cast<uint32_t>(Z >> 32);
    // two orders of the same additions; measured with 384 threads per block: the first is 3 % faster for E2M1 and 3 %
    // slower for E4M3; with 512 threads the two are within 0.5 % of each other for both formats
    if (FMT == kE2M1) return ((eqbits >> (23 - F::M)) + zhi) + (r < zlo ? 1u - kBase : 0u - kBase);
    return (eqbits >> (23 - F::M)) + (zhi - kBase + (r < zlo ? 1u : 0u));
}

// one FP8 byte (E4M3 / E5M2): NaN -> 0x7F without a sign, E5M2 keeps infinity
template <int FMT>
__device__ __forceinline__ uint32_t sr_fp8_code(uint32_t fbits, uint32_t r) {
    const float x = __uint_as_float(fbits);
    uint32_t code = min(sr_small_magnitude<FMT, true>(x, r), 0x7Fu);
    if (FMT == kE5M2) code = fabsf(x) == __uint_as_float(0x7F800000u) ? kE5M2InfCode : code;
    return code == 0x7Fu ? code : (code | ((fbits >> 24) & 0x80u));
}

// E2M1: sign in bit 3 (kept for NaN too), magnitude code in bits 0..2
__device__ __forceinline__ uint32_t sr_fp4_code(uint32_t fbits, uint32_t r) {
    return ((fbits >> 28) & 8u) | sr_small_magnitude<kE2M1, false>(__uint_as_float(fbits), r);
}

// four values -> four 4-bit codes in bits 0..15 (element j in bits 4j..4j+3)
__device__ __forceinline__ uint32_t cast4_fp4(const uint4 x, const uint4 w) {
    const uint32_t n0 = sr_fp4_code(x.x, w.x), n1 = sr_fp4_code(x.y, w.y), n2 = sr_fp4_code(x.z, w.z), n3 = sr_fp4_code(x.w, w.w);
    // shift-adds on the ALU pipe: this kernel has the FMA pipe fuller than the FP8 one (0.295 -> 0.288 ms)
    return (n1 * 16u + n0) + (n3 * 16u + n2) * 256u;
}

__device__ __forceinline__ uint32_t noise32_of_element(uint64_t idx, uint32_t c2, uint32_t c3, const PhiloxKeys& K) {
    const uint64_t number = idx >> 2;
    const uint4 w = philox4x32_10(static_cast<uint32_t>(number), static_cast<uint32_t>(number >> 32), c2, c3, K);
    const uint32_t e = static_cast<uint32_t>(idx) & 3u;
    return e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w;
}

// four values -> four bytes; the four sign bits are gathered with byte permutes
template <int FMT>
__device__ __forceinline__ uint32_t cast4(const uint4 x, const uint4 w) {
    const float f0 = __uint_as_float(x.x), f1 = __uint_as_float(x.y), f2 = __uint_as_float(x.z), f3 = __uint_as_float(x.w);
    uint32_t m0 = min(sr_small_magnitude<FMT, true>(f0, w.x), 0x7Fu), m1 = min(sr_small_magnitude<FMT, true>(f1, w.y), 0x7Fu);
    uint32_t m2 = min(sr_small_magnitude<FMT, true>(f2, w.z), 0x7Fu), m3 = min(sr_small_magnitude<FMT, true>(f3, w.w), 0x7Fu);
    if (FMT == kE5M2) {
        const float inf = __uint_as_float(0x7F800000u);
        m0 = fabsf(f0) == inf ? kE5M2InfCode : m0;
        m1 = fabsf(f1) == inf ? kE5M2InfCode : m1;
        m2 = fabsf(f2) == inf ? kE5M2InfCode : m2;
        m3 = fabsf(f3) == inf ? kE5M2InfCode : m3;
    }
    const uint32_t mags = (m1 * mul_256() + m0) + (m3 * mul_256() + m2) * mul_65536();   // on the FMA pipe (0.325 -> 0.321 ms)
    const uint32_t tops = __byte_perm(__byte_perm(x.x, x.y, 0x0073), __byte_perm(x.z, x.w, 0x0073), 0x5410);
    // a NaN code (0x7F) keeps no sign: every magnitude byte is at most 0x7F, so adding 1 to each sets its bit 7
    // exactly where it is 0x7F
    const uint32_t nan7 = mags + 0x01010101u;
    return mags | (tops & ~nan7 & 0x80808080u);
}

// sixteen consecutive values -> sixteen bytes (four Philox calls)
template <int FMT>
__device__ __forceinline__ uint4 cast16(const float* __restrict__ src, uint64_t vec, uint64_t elem_offset, uint32_t c1, uint32_t tensor_id,
                                        uint32_t seed_hi, const PhiloxKeys& K) {
    const uint4 a = ld16(src, 4 * vec), b = ld16(src, 4 * vec + 1), c = ld16(src, 4 * vec + 2), d = ld16(src, 4 * vec + 3);
    const uint64_t number = (elem_offset + (vec << 4)) >> 2;
    const uint32_t c0 = static_cast<uint32_t>(number);
    uint4 o;
    o.x = cast4<FMT>(a, philox4x32_10(c0, c1, tensor_id, seed_hi, K));
    o.y = cast4<FMT>(b, philox4x32_10(c0 + 1, c1, tensor_id, seed_hi, K));
    o.z = cast4<FMT>(c, philox4x32_10(c0 + 2, c1, tensor_id, seed_hi, K));
    o.w = cast4<FMT>(d, philox4x32_10(c0 + 3, c1, tensor_id, seed_hi, K));
    return o;
}

// sixteen consecutive values -> sixteen 4-bit codes in eight bytes
__device__ __forceinline__ uint2 cast16_fp4(const float* __restrict__ src, uint64_t vec, uint64_t elem_offset, uint32_t c1, uint32_t tensor_id,
                                            uint32_t seed_hi, const PhiloxKeys& K) {
    const uint4 a = ld16(src, 4 * vec), b = ld16(src, 4 * vec + 1), c = ld16(src, 4 * vec + 2), d = ld16(src, 4 * vec + 3);
    const uint64_t number = (elem_offset + (vec << 4)) >> 2;
    const uint32_t c0 = static_cast<uint32_t>(number);
    const uint32_t lo = cast4_fp4(a, philox4x32_10(c0, c1, tensor_id, seed_hi, K)) |
                        (cast4_fp4(b, philox4x32_10(c0 + 1, c1, tensor_id, seed_hi, K)) << 16);
    const uint32_t hi = cast4_fp4(c, philox4x32_10(c0 + 2, c1, tensor_id, seed_hi, K)) |
                        (cast4_fp4(d, philox4x32_10(c0 + 3, c1, tensor_id, seed_hi, K)) << 16);
    return make_uint2(lo, hi);
}

// Up to 128 registers: the values of an iteration are independent and the two pipes overlap only when the compiler
// may keep several of them in flight.  E4M3, same GPU: 16 values per iteration with 40 registers 0.321 ms, with 72
// registers 0.299-0.313 ms; 32 values per iteration with 109-122 registers 0.300-0.306 ms; 4 or 8 values per
// iteration with two to four times the resident warps 0.33-0.42 ms.  One block per SM, threads per block (2^28
// values, E4M3 / E2M1, same GPU): 256 0.293 / 0.280, 384 0.294 / 0.278, 512 0.282 / 0.275, 640 0.288 / 0.273,
// 768 0.290 / 0.275, 1024 0.294 / 0.283 ms; two blocks of 192 0.309 / 0.294, four of 128 0.306 / 0.293 ms.
constexpr int kSmallThreads = 512;
constexpr int kSmallMinBlocks = 1;

// VEC: 16 elements per thread-iteration (4 x 16-byte loads, 1 x 16-byte store); needs both buffers
// 16-byte aligned, elem_offset a multiple of 16 and every index of the launch's whole vectors with the same
// (index >> 34), the high word c1 of the call number: the first Philox round's product with the tensor id and what
// follows from it and c1 alone are then loop-invariant (E2M1 0.282 -> 0.277 ms).
template <int FMT, bool VEC>
__global__ void __launch_bounds__(kSmallThreads, kSmallMinBlocks)
k_sr_downcast_fp8(const float* __restrict__ src, uint8_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
                  uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (VEC) {
        const uint64_t nvec = n >> 4;
        const uint32_t c1 = static_cast<uint32_t>(elem_offset >> 34);
        // two vectors per iteration: 32 independent values for the compiler to interleave
        uint64_t vec = tid;
        for (; vec + stride < nvec; vec += 2 * stride) {
            const uint4 o0 = cast16<FMT>(src, vec, elem_offset, c1, tensor_id, seed_hi, K);
            const uint4 o1 = cast16<FMT>(src, vec + stride, elem_offset, c1, tensor_id, seed_hi, K);
            st16(dst, vec, o0);
            st16(dst, vec + stride, o1);
        }
        if (vec < nvec) st16(dst, vec, cast16<FMT>(src, vec, elem_offset, c1, tensor_id, seed_hi, K));
        done = nvec << 4;
    }
    for (uint64_t i = done + tid; i < n; i += stride)
        dst[i] = static_cast<uint8_t>(sr_fp8_code<FMT>(__float_as_uint(src[i]), noise32_of_element(elem_offset + i, tensor_id, seed_hi, K)));
}

// E2M1, two codes per byte (element 2j in bits 0..3 of byte j).  VEC: 16 elements per
// thread-iteration (4 x 16-byte loads, one 8-byte store); needs src 16-byte and dst 8-byte aligned,
// elem_offset a multiple of 16 and one (index >> 34) for the launch's whole vectors.  The rest (and everything without VEC) goes byte by byte, one
// thread per output byte.
template <bool VEC>
__global__ void __launch_bounds__(kSmallThreads, kSmallMinBlocks)
k_sr_downcast_fp4(const float* __restrict__ src, uint8_t* __restrict__ dst, uint64_t n, uint64_t elem_offset,
                  uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K) {
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t done = 0;
    if (VEC) {
        const uint64_t nvec = n >> 4;
        const uint32_t c1 = static_cast<uint32_t>(elem_offset >> 34);
        // two vectors per iteration: 32 independent values for the compiler to interleave
        uint64_t vec = tid;
        for (; vec + stride < nvec; vec += 2 * stride) {
            const uint2 o0 = cast16_fp4(src, vec, elem_offset, c1, tensor_id, seed_hi, K);
            const uint2 o1 = cast16_fp4(src, vec + stride, elem_offset, c1, tensor_id, seed_hi, K);
            __stcs(reinterpret_cast<uint2*>(dst) + vec, o0);
            __stcs(reinterpret_cast<uint2*>(dst) + vec + stride, o1);
        }
        if (vec < nvec) __stcs(reinterpret_cast<uint2*>(dst) + vec, cast16_fp4(src, vec, elem_offset, c1, tensor_id, seed_hi, K));
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

// length of the next launch of a vector-path call: up to the next multiple of 2^34 (one c1 per launch)
inline uint64_t next_small_launch(uint64_t idx, uint64_t left) {
    const uint64_t to_boundary = (static_cast<uint64_t>(1) << 34) - (idx & ((static_cast<uint64_t>(1) << 34) - 1));
    return left < to_boundary ? left : to_boundary;
}

template <int FMT, bool VEC>
cudaError_t launch_fp8_t(const float* src, uint8_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                         uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream) {
    auto k = k_sr_downcast_fp8<FMT, VEC>;
    for (uint64_t done = 0; done < n;) {
        const uint64_t len = VEC ? next_small_launch(elem_offset + done, n - done) : n;
        const uint64_t items = VEC ? (len >> 4) + 16 : len;
        k<<<grid_for(k, items, dev, kSmallThreads), kSmallThreads, 0, stream>>>(src + done, dst + done, len, elem_offset + done,
                                                                                tensor_id, seed_hi, K);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        done += len;
    }
    return cudaSuccess;
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
    if (!vec) {
        auto k = k_sr_downcast_fp4<false>;
        k<<<grid_for(k, (n + 1) >> 1, dev, kSmallThreads), kSmallThreads, 0, stream>>>(src, dst, n, elem_offset, tensor_id, seed_hi, K);
        return cudaGetLastError();
    }
    auto k = k_sr_downcast_fp4<true>;
    // a cut falls on a multiple of 16 elements: whole vectors and whole bytes before it
    for (uint64_t done = 0; done < n;) {
        const uint64_t len = next_small_launch(elem_offset + done, n - done);
        k<<<grid_for(k, (len >> 4) + 16, dev, kSmallThreads), kSmallThreads, 0, stream>>>(src + done, dst + (done >> 1), len,
                                                                                          elem_offset + done, tensor_id, seed_hi, K);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        done += len;
    }
    return cudaSuccess;
}

}  // namespace sradamw
