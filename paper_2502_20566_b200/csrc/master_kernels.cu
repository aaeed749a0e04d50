// FP32-master mixed-precision AdamW: the recipe the paper compares against (FP32 master weights and
// FP32 moments, BF16 copy of the weights for the forward pass).  Same element function as the SR
// step, no noise; x, m, v stay FP32 and x is also written as nearest-rounded BF16 (Eq. 1).
// 28 bytes per element with BF16 gradients (12 + 2 read, 12 + 2 written), 30 with FP32 gradients:
// twice the traffic of the BF16+SR step, which is what the comparison is for.

#include "adamw_body.cuh"

namespace sradamw {

namespace {

__device__ __forceinline__ float4 ldf4(const float* base, uint64_t i4) {
    const uint4 r = __ldcs(reinterpret_cast<const uint4*>(base) + i4);
    return make_float4(__uint_as_float(r.x), __uint_as_float(r.y), __uint_as_float(r.z), __uint_as_float(r.w));
}
__device__ __forceinline__ void stf4(float* base, uint64_t i4, float a, float b, float c, float d) {
    __stcs(reinterpret_cast<uint4*>(base) + i4,
           make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d)));
}

__device__ __forceinline__ uint32_t rne_pair(float even, float odd) {
    const uint32_t a = __float_as_uint(even), b = __float_as_uint(odd);
    const uint32_t sa = is_nan_bits(a) ? (kQuietNaNbf16 << 16) : rne_sum(a);
    const uint32_t sb = is_nan_bits(b) ? (kQuietNaNbf16 << 16) : rne_sum(b);
    return pack_top_halves(sa, sb);
}

template <bool G32>
__device__ __forceinline__ void master_scalar(float* p, uint16_t* p16, const void* g, float* m, float* v, uint64_t i,
                                              float gscale, const StepScalars& S) {
    const float gi = G32 ? static_cast<const float*>(g)[i]
                         : __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(g)[i]) << 16);
    const ElementOut r = adamw_element(p[i], gi, m[i], v[i], gscale, S);
    p[i] = r.x;
    m[i] = r.m;
    v[i] = r.v;
    const uint32_t b = __float_as_uint(r.x);
    p16[i] = static_cast<uint16_t>((is_nan_bits(b) ? (kQuietNaNbf16 << 16) : rne_sum(b)) >> 16);
}

// Eight consecutive elements per thread-iteration: 6 x 16-byte loads for x, m, v, one or two for g;
// 6 x 16-byte stores and one for the BF16 copy.  FAST: branch-free arithmetic inside the validated
// operand range with the reference arithmetic as fallback for the vector, as in the SR kernels.
// WIDE: x, m, v (and FP32 g) are 32-byte aligned and move with one 32-byte access per thread and
// array (measured on B200: 84 % -> 94 % of the copy peak on 832M elements).
template <bool G32, bool FAST, int VAR, bool WIDE>
__global__ void __launch_bounds__(kBlockThreads, 4)
k_master_adamw(float* p, uint16_t* p16, const void* g, float* m, float* v, uint64_t n, bool vec_ok,
               const __grid_constant__ StepScalars S) {
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    if (!vec_ok) {
        for (uint64_t i = tid; i < n; i += stride) master_scalar<G32>(p, p16, g, m, v, i, gscale, S);
        return;
    }
    const uint64_t nvec = n >> 3;
    for (uint64_t vec = tid; vec < nvec; vec += stride) {
        float x[8], mm[8], vv[8], ge[8];
        if (WIDE) {
            const Words8 pw = ld32(p, vec), mw = ld32(m, vec), vw = ld32(v, vec);
            load_grad8<G32>(g, vec, ge, true);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                x[e] = __uint_as_float(pw.w[e]);
                mm[e] = __uint_as_float(mw.w[e]);
                vv[e] = __uint_as_float(vw.w[e]);
            }
        } else {
            const float4 pa = ldf4(p, 2 * vec), pb = ldf4(p, 2 * vec + 1);
            const float4 ma = ldf4(m, 2 * vec), mb = ldf4(m, 2 * vec + 1);
            const float4 va = ldf4(v, 2 * vec), vb = ldf4(v, 2 * vec + 1);
            load_grad8<G32>(g, vec, ge);
            const float xs[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
            const float ms[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
            const float vs[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                x[e] = xs[e];
                mm[e] = ms[e];
                vv[e] = vs[e];
            }
        }
        ElementOut r[8];
        bool redo = !FAST;
        if (FAST) {
            RangeTrack track;
            track.init();
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                r[e] = adamw_element_in_range<VAR>(x[e], ge[e], mm[e], vv[e], gscale, S);
                r[e + 1] = adamw_element_in_range<VAR>(x[e + 1], ge[e + 1], mm[e + 1], vv[e + 1], gscale, S);
                track.add(r[e], r[e + 1]);
            }
            redo = track.left_range();
        }
        if (redo) {
#pragma unroll
            for (int e = 0; e < 8; ++e) r[e] = adamw_element(x[e], ge[e], mm[e], vv[e], gscale, S);
        }
        if (WIDE) {
            Words8 xo, mo, vo;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                xo.w[e] = __float_as_uint(r[e].x);
                mo.w[e] = __float_as_uint(r[e].m);
                vo.w[e] = __float_as_uint(r[e].v);
            }
            st32(p, vec, xo);
            st32(m, vec, mo);
            st32(v, vec, vo);
        } else {
            stf4(p, 2 * vec, r[0].x, r[1].x, r[2].x, r[3].x);
            stf4(p, 2 * vec + 1, r[4].x, r[5].x, r[6].x, r[7].x);
            stf4(m, 2 * vec, r[0].m, r[1].m, r[2].m, r[3].m);
            stf4(m, 2 * vec + 1, r[4].m, r[5].m, r[6].m, r[7].m);
            stf4(v, 2 * vec, r[0].v, r[1].v, r[2].v, r[3].v);
            stf4(v, 2 * vec + 1, r[4].v, r[5].v, r[6].v, r[7].v);
        }
        st16(p16, vec, make_uint4(rne_pair(r[0].x, r[1].x), rne_pair(r[2].x, r[3].x), rne_pair(r[4].x, r[5].x),
                                  rne_pair(r[6].x, r[7].x)));
    }
    const uint64_t done = nvec << 3;
    if (tid < n - done) master_scalar<G32>(p, p16, g, m, v, done + tid, gscale, S);
}

template <bool G32, bool FAST, int VAR, bool WIDE>
cudaError_t launch_master_w(float* p, uint16_t* p16, const void* g, float* m, float* v, uint64_t n, bool vec_ok,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    auto k = k_master_adamw<G32, FAST, VAR, WIDE>;
    const uint64_t items = vec_ok ? (n >> 3) + 8 : n;
    k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(p, p16, g, m, v, n, vec_ok, S);
    return cudaGetLastError();
}

template <bool G32, bool FAST, int VAR>
cudaError_t launch_master_t(float* p, uint16_t* p16, const void* g, float* m, float* v, uint64_t n, bool vec_ok,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    auto aligned32 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 31u) == 0; };
    const bool wide = vec_ok && aligned32(p) && aligned32(m) && aligned32(v) && (!G32 || aligned32(g));
    return wide ? launch_master_w<G32, FAST, VAR, true>(p, p16, g, m, v, n, vec_ok, S, dev, stream)
                : launch_master_w<G32, FAST, VAR, false>(p, p16, g, m, v, n, vec_ok, S, dev, stream);
}

}  // namespace

cudaError_t launch_master_adamw(float* p, uint16_t* p16, const void* g, bool g_f32, float* m, float* v, uint64_t n,
                                const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    const bool vec_ok = aligned16(p) && aligned16(p16) && aligned16(g) && aligned16(m) && aligned16(v);
    const bool fast = fast_path_allowed(S), scale = needs_scale(S);
#define SR_M(G, F, VARIANT) launch_master_t<G, F, VARIANT>(p, p16, g, m, v, n, vec_ok, S, dev, stream)
    // VARIANT: bit 0 gradient scale, bit 1 epsilon under the square root (fast arithmetic only)
    const int var = (scale ? 1 : 0) | (S.eps_inside ? 2 : 0);
    if (g_f32) {
        if (!fast) return SR_M(true, false, 1);
        switch (var) {
            case 0: return SR_M(true, true, 0);
            case 1: return SR_M(true, true, 1);
            case 2: return SR_M(true, true, 2);
            default: return SR_M(true, true, 3);
        }
    }
    if (!fast) return SR_M(false, false, 1);
    switch (var) {
        case 0: return SR_M(false, true, 0);
        case 1: return SR_M(false, true, 1);
        case 2: return SR_M(false, true, 2);
        default: return SR_M(false, true, 3);
    }
#undef SR_M
}

}  // namespace sradamw
