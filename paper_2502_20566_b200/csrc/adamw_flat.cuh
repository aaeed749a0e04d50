// Flat-buffer kernel of the fused SR-AdamW step and its launcher, for one gradient type.
#pragma once

#include <atomic>

#include "adamw_body.cuh"

// Direct-load shape (FP32 gradients): the next vector's loads are issued before the current vector is
// computed.  Measured on B200, 832M elements, same GPU: 2.26 -> 2.15 ms.
#ifndef SR_DIRECT_PREFETCH
#define SR_DIRECT_PREFETCH 1
#endif

namespace sradamw {

// MODE 0: element-wise (any alignment, any offset)
//      1: 16-byte vectors, reference arithmetic, elem_offset not a multiple of 8: every vector straddles two
//         noise groups (six Philox calls per vector)
//      4: 16-byte vectors, reference arithmetic, one Philox call per (vector, slot): elem_offset a
//         multiple of 8 but scalars outside what the branch-free arithmetic covers (beta2 so close to 1 that
//         1/sqrt(1 - beta2^t) > 1024, eps > 1)
// Persistent grid: thread t takes vectors t, t + T, t + 2T, ... (T = threads in the grid).
template <bool G32, uint32_t FLAGS, int MODE>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocksPerSM)
k_sr_adamw_flat(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
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
    for (uint64_t vec = tid; vec < nvec; vec += stride)
        step_vec8_reference<G32, FLAGS, MODE == 4>(p, g, m, v, vec, elem_offset + (vec << 3), tensor_id, seed_hi, gscale, K, S);
    const uint64_t done = nvec << 3;
    if (tid < n - done)
        step_scalar<G32, FLAGS>(p, g, m, v, done + tid, elem_offset + done + tid, tensor_id, seed_hi, gscale, K, S);
}

// The hot kernel (modes 2 and 3 of the launcher): 16-byte vectors, branch-free arithmetic, gradient
// used as is or multiplied by gscale (VAR bit 0), epsilon outside or under the square root (VAR bit 1).
// VAR bit 2: elem_offset is not a multiple of 8 (noise exchanged between lanes).  Every
// index of the launch has the same (index >> 33) = c1.  Same persistent grid.  STAGED = true: each
// thread keeps its next vectors in flight -- while vector k is computed out of shared memory, the
// asynchronous copies of vectors k + T, ... are already under way (kFlatStages slots per thread and
// array).  SHAPE 0: direct loads into registers, kFlatDirectThreads x kFlatDirectMinBlocks (FP32 gradients); 2: staged,
// kFlatStagedThreads x kFlatStagedMinBlocks, kFlatStages (BF16 gradients, every launch length).
template <bool G32, uint32_t FLAGS, int VAR, int SHAPE>
__global__ void __launch_bounds__(SHAPE == 2 ? (G32 ? kFlatStagedThreadsF32 : kFlatStagedThreads) : kFlatDirectThreads,
                                  SHAPE == 2 ? kFlatStagedMinBlocks : kFlatDirectMinBlocks)
k_sr_adamw_flat_fast(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                     uint32_t c1, uint32_t tensor_id, uint32_t seed_hi, const __grid_constant__ PhiloxKeys K,
                     const __grid_constant__ StepScalars S) {
    // FP32 gradients: x, m, v are staged, the gradient's two 16-byte pieces are loaded straight into a register double
    // buffer (five staged pieces per vector measured slower than no staging at all, three staged + two direct faster)
    constexpr bool kHybrid = G32 && (VAR & 4) == 0;
    constexpr int kArrays = kHybrid ? 3 : G32 ? 5 : 4;   // staged 16-byte pieces per vector
    constexpr bool STAGED = SHAPE != 0;
    constexpr int kThreads = SHAPE == 2 ? (G32 ? kFlatStagedThreadsF32 : kFlatStagedThreads) : kFlatDirectThreads;
    static_assert(SHAPE == 0 || SHAPE == 2, "direct or staged");
    constexpr int kStages = G32 ? kFlatStagesF32 : kFlatStages;
    // The staging (and, with straddling vectors, the table of head calls) is more than the 48 KB a kernel gets
    // without asking: it lives in dynamic shared memory that the launcher sizes.
    constexpr bool kDynamic = STAGED;
    constexpr int kStageEntries = STAGED ? kStages * kArrays * kThreads : 1;
    extern __shared__ uint4 dynamic_smem[];
    uint4* const stage = dynamic_smem;
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    const uint64_t nvec = n >> 3;
    if constexpr ((VAR & 4) != 0) {
        // elem_offset is not a multiple of 8: every vector straddles two noise groups.  Same grid-stride walk over
        // rows of 32 vectors as below; every lane computes the calls of the group its vector ends in and receives
        // those of the group it starts in from the lane below (RowChain): three calls per vector as in the
        // aligned case, plus 3/32 for the head calls.  The loop is uniform over the warp (the shuffles need every
        // lane) and covers whole rows only; the vectors of the last, partial row go element by element with the
        // ragged tail.
        using Chain = RowChain<FLAGS & 7u, true>;
        __shared__ uint4 heads_static[kDynamic ? 1 : (kThreads / 32) * Chain::kTableEntries];
        uint4* const heads = kDynamic ? dynamic_smem + kStageEntries : heads_static;
        const uint32_t lane = threadIdx.x & 31u;
        const Chain chain{heads + (threadIdx.x >> 5) * Chain::kTableEntries, elem_offset >> 3, stride,
                          static_cast<uint32_t>(elem_offset) & 7u, lane, c1, tensor_id, seed_hi};
        const uint64_t row_vecs = nvec & ~static_cast<uint64_t>(31);      // vectors in whole rows
        uint32_t k = 0;
        auto noise = [&](uint64_t vec, uint4& wx, uint4& wm, uint4& wv) {
            if ((k & 31u) == 0u) chain.refill(vec - lane, K);
            uint4 w[4];
            chain.words(vec, k, K, w);
            ++k;
            if (FLAGS & 1u) wx = w[0];
            if (FLAGS & 2u) wm = w[1];
            if (FLAGS & 4u) wv = w[2];
        };
        if (STAGED) {
            uint4* const mine = stage + threadIdx.x;
            auto slot = [&](int s, int a) -> uint4* { return mine + (s * kArrays + a) * kThreads; };
            auto issue = [&](uint64_t vec, int s) {
                if (vec < row_vecs) {
                    async_copy16(slot(s, 0), reinterpret_cast<const uint4*>(p) + vec);
                    async_copy16(slot(s, 1), reinterpret_cast<const uint4*>(m) + vec);
                    async_copy16(slot(s, 2), reinterpret_cast<const uint4*>(v) + vec);
                    if (G32) {
                        async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(g) + 2 * vec);
                        async_copy16(slot(s, 4), reinterpret_cast<const uint4*>(g) + 2 * vec + 1);
                    } else {
                        async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(g) + vec);
                    }
                }
                async_copy_commit();
            };
#pragma unroll
            for (int s = 0; s < kStages - 1; ++s) issue(tid + s * stride, s);
            int s = 0;
            for (uint64_t vec = tid; vec < row_vecs; vec += stride) {
                int ahead = s + kStages - 1;
                if (ahead >= kStages) ahead -= kStages;
                issue(vec + (kStages - 1) * stride, ahead);
                uint4 wx = make_uint4(0, 0, 0, 0), wm = wx, wv = wx;
                noise(vec, wx, wm, wv);
                async_copy_wait<kStages - 1>();
                const uint4 pv = *slot(s, 0), mv = *slot(s, 1), vv = *slot(s, 2);
                float ge[8];
                unpack_grad8<G32>(*slot(s, 3), G32 ? *slot(s, kArrays - 1) : make_uint4(0, 0, 0, 0), ge);
                step_vec8_fast_noise<G32, FLAGS, VAR>(p, g, m, v, vec, elem_offset + (vec << 3), pv, mv, vv, ge, wx, wm, wv,
                                                        tensor_id, seed_hi, gscale, K, S);
                if (++s == kStages) s = 0;
            }
            async_copy_wait<0>();
        } else {
            uint4 pv = make_uint4(0, 0, 0, 0), mv = pv, vv = pv, g0 = pv, g1 = pv;
            auto load = [&](uint64_t vec, uint4& a, uint4& b, uint4& c, uint4& d0, uint4& d1) {
                if (vec < row_vecs) {
                    a = ld16(p, vec);
                    b = ld16(m, vec);
                    c = ld16(v, vec);
                    if (G32) {
                        d0 = ld16(g, 2 * vec);
                        d1 = ld16(g, 2 * vec + 1);
                    } else {
                        d0 = ld16(g, vec);
                    }
                }
            };
            load(tid, pv, mv, vv, g0, g1);
            for (uint64_t vec = tid; vec < row_vecs; vec += stride) {
                uint4 pn = pv, mn = mv, vn = vv, gn0 = g0, gn1 = g1;
                load(vec + stride, pn, mn, vn, gn0, gn1);
                uint4 wx = make_uint4(0, 0, 0, 0), wm = wx, wv = wx;
                noise(vec, wx, wm, wv);
                float ge[8];
                unpack_grad8<G32>(g0, g1, ge);
                step_vec8_fast_noise<G32, FLAGS, VAR>(p, g, m, v, vec, elem_offset + (vec << 3), pv, mv, vv, ge, wx, wm, wv,
                                                        tensor_id, seed_hi, gscale, K, S);
                pv = pn; mv = mn; vv = vn; g0 = gn0; g1 = gn1;
            }
        }
    } else if (STAGED) {
        uint4* const mine = stage + threadIdx.x;
        auto slot = [&](int s, int a) -> uint4* { return mine + (s * kArrays + a) * kThreads; };
        auto issue = [&](uint64_t vec, int s) {
            if (vec < nvec) {
                async_copy16(slot(s, 0), reinterpret_cast<const uint4*>(p) + vec);
                async_copy16(slot(s, 1), reinterpret_cast<const uint4*>(m) + vec);
                async_copy16(slot(s, 2), reinterpret_cast<const uint4*>(v) + vec);
                if (kHybrid) {
                } else if (G32) {
                    async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(g) + 2 * vec);
                    async_copy16(slot(s, 4), reinterpret_cast<const uint4*>(g) + 2 * vec + 1);
                } else {
                    async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(g) + vec);
                }
            }
            async_copy_commit();   // one group per iteration, empty past the end: the wait count stays uniform
        };
#pragma unroll
        for (int s = 0; s < kStages - 1; ++s) issue(tid + s * stride, s);
        int s = 0;
        uint4 g0 = make_uint4(0, 0, 0, 0), g1 = g0;
        if (kHybrid && tid < nvec) {
            g0 = ld16(g, 2 * tid);
            g1 = ld16(g, 2 * tid + 1);
        }
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            int ahead = s + kStages - 1;
            if (ahead >= kStages) ahead -= kStages;
            issue(vec + (kStages - 1) * stride, ahead);
            uint4 gn0 = g0, gn1 = g1;
            if (kHybrid && vec + stride < nvec) {
                gn0 = ld16(g, 2 * (vec + stride));
                gn1 = ld16(g, 2 * (vec + stride) + 1);
            }
            async_copy_wait<kStages - 1>();   // this vector's group has landed
            const uint4 pv = *slot(s, 0), mv = *slot(s, 1), vv = *slot(s, 2);
            float ge[8];
            if (kHybrid) unpack_grad8<true>(g0, g1, ge);
            else unpack_grad8<G32>(*slot(s, kHybrid ? 0 : 3), G32 ? *slot(s, kArrays - 1) : make_uint4(0, 0, 0, 0), ge);
            g0 = gn0; g1 = gn1;
            step_vec8_fast_loaded<G32, FLAGS, VAR>(p, g, m, v, vec, elem_offset + (vec << 3), pv, mv, vv, ge, c1,
                                                     tensor_id, seed_hi, gscale, K, S);
            if (++s == kStages) s = 0;
        }
        async_copy_wait<0>();
    } else {
#if SR_DIRECT_PREFETCH
        // the next vector's loads are issued before the current one is computed (register double buffer)
        uint4 pv = make_uint4(0, 0, 0, 0), mv = pv, vv = pv, g0 = pv, g1 = pv;
        auto load = [&](uint64_t vec, uint4& a, uint4& b, uint4& c, uint4& d0, uint4& d1) {
            if (vec < nvec) {
                a = ld16(p, vec);
                b = ld16(m, vec);
                c = ld16(v, vec);
                if (G32) {
                    d0 = ld16(g, 2 * vec);
                    d1 = ld16(g, 2 * vec + 1);
                } else {
                    d0 = ld16(g, vec);
                }
            }
        };
        load(tid, pv, mv, vv, g0, g1);
        for (uint64_t vec = tid; vec < nvec; vec += stride) {
            uint4 pn = pv, mn = mv, vn = vv, gn0 = g0, gn1 = g1;
            load(vec + stride, pn, mn, vn, gn0, gn1);
            float ge[8];
            unpack_grad8<G32>(g0, g1, ge);
            step_vec8_fast_loaded<G32, FLAGS, VAR>(p, g, m, v, vec, elem_offset + (vec << 3), pv, mv, vv, ge, c1, tensor_id, seed_hi,
                                                     gscale, K, S);
            pv = pn; mv = mn; vv = vn; g0 = gn0; g1 = gn1;
        }
#else
        for (uint64_t vec = tid; vec < nvec; vec += stride)
            step_vec8_fast<G32, FLAGS, VAR>(p, g, m, v, vec, elem_offset + (vec << 3), c1, tensor_id, seed_hi, gscale, K, S);
#endif
    }
    // ragged tail; with straddling vectors also the last, partial row (fewer than 32 * 8 + 8 elements)
    const uint64_t done = ((VAR & 4) != 0 ? nvec & ~static_cast<uint64_t>(31) : nvec) << 3;
    for (uint64_t i = done + tid; i < n; i += stride)
        step_scalar<G32, FLAGS>(p, g, m, v, i, elem_offset + i, tensor_id, seed_hi, gscale, K, S);
}

// Which gradient types use the staged variant.  Measured on B200 (same GPU, back to back): BF16
// gradients 85.3% staged vs 83.8% direct of the copy peak at 6.7B (in the block shapes of that time); FP32
// gradients with all five 16-byte pieces of a vector staged 77.7% vs 93.2% direct at 832M elements, with x, m, v
// staged and the gradient loaded directly 98.7%.
#ifndef SR_STAGE_BF16
#define SR_STAGE_BF16 1
#endif
#ifndef SR_STAGE_F32
#define SR_STAGE_F32 1
#endif

template <bool G32, uint32_t FLAGS, int MODE, bool EPS_IN = false, bool STRADDLE = false>
cudaError_t launch_flat_mode(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                             uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S,
                             const DeviceInfo& dev, cudaStream_t stream) {
    // + 8: enough threads for the ragged tail
    const uint64_t items = MODE == 0 ? n : (n >> 3) + 8;
    if (MODE == 2 || MODE == 3) {
        constexpr bool kStaged = G32 ? (SR_STAGE_F32 != 0 && !STRADDLE) : (SR_STAGE_BF16 != 0);
        const uint32_t c1 = static_cast<uint32_t>(elem_offset >> 33);
        constexpr int kVar = (MODE == 3 ? 1 : 0) | (EPS_IN ? 2 : 0) | (STRADDLE ? 4 : 0);
        if constexpr (kStaged) {
            auto k = k_sr_adamw_flat_fast<G32, FLAGS, kVar, 2>;
            // staging, plus one table of head calls per warp where vectors straddle noise groups: more than the 48 KB a
            // kernel gets without asking
            constexpr int kThreads = G32 ? kFlatStagedThreadsF32 : kFlatStagedThreads;
            const size_t dynamic = sizeof(uint4) * ((G32 ? kFlatStagesF32 * 3 : kFlatStages * 4) * kThreads +
                                                    (STRADDLE ? (kThreads / 32) * RowChain<FLAGS & 7u, true>::kTableEntries : 0));
            static std::atomic<int> prepared[kMaxDevices] = {};      // per kernel instantiation and device
            if (!prepared[dev.index].load(std::memory_order_acquire)) {
                const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(dynamic));
                if (e != cudaSuccess) return e;
                prepared[dev.index].store(1, std::memory_order_release);
            }
            k<<<grid_for(k, items, dev, kThreads, dynamic), kThreads, dynamic, stream>>>(
                p, g, m, v, n, elem_offset, c1, tensor_id, seed_hi, K, S);
        } else {
            auto k = k_sr_adamw_flat_fast<G32, FLAGS, kVar, 0>;
            k<<<grid_for(k, items, dev, kFlatDirectThreads), kFlatDirectThreads, 0, stream>>>(p, g, m, v, n, elem_offset, c1, tensor_id,
                                                                                                 seed_hi, K, S);
        }
    } else {
        auto k = k_sr_adamw_flat<G32, FLAGS, (MODE < 2 || MODE == 4 ? MODE : 0)>;
        k<<<grid_for(k, items, dev), kBlockThreads, 0, stream>>>(p, g, m, v, n, elem_offset, tensor_id, seed_hi, K, S);
    }
    return cudaGetLastError();
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_flat_flags(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                              uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const StepScalars& S,
                              const DeviceInfo& dev, cudaStream_t stream) {
    const size_t gsz = G32 ? 4 : 2;
    // launches of at most 1.5 * kFlatLaunchElems elements, none of which crosses a multiple of 2^33 in global index
    // space (every index of a launch shares index >> 33)
    uint64_t done = 0;
    while (done < n) {
        const uint64_t idx = elem_offset + done;
        const uint64_t len = next_flat_launch(idx, n - done);
        uint16_t* ps = p + done;
        const void* gs = static_cast<const char*>(g) + done * gsz;
        uint16_t* ms = m + done;
        uint16_t* vs = v + done;
        const bool vec = aligned16(ps) && aligned16(gs) && aligned16(ms) && aligned16(vs);
        cudaError_t e;
        if (!vec)
            e = launch_flat_mode<G32, FLAGS, 0>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if ((idx & 7u) != 0 && !fast_path_allowed(S))
            e = launch_flat_mode<G32, FLAGS, 1>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if ((idx & 7u) != 0)   // branch-free arithmetic, every vector straddling two noise groups
            e = S.eps_inside ? (needs_scale(S) ? launch_flat_mode<G32, FLAGS, 3, true, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream)
                                               : launch_flat_mode<G32, FLAGS, 2, true, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream))
                             : (needs_scale(S) ? launch_flat_mode<G32, FLAGS, 3, false, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream)
                                               : launch_flat_mode<G32, FLAGS, 2, false, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream));
        else if (!fast_path_allowed(S))
            e = launch_flat_mode<G32, FLAGS, 4>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if (S.eps_inside && needs_scale(S))
            e = launch_flat_mode<G32, FLAGS, 3, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
        else if (S.eps_inside)
            e = launch_flat_mode<G32, FLAGS, 2, true>(ps, gs, ms, vs, len, idx, tensor_id, seed_hi, K, S, dev, stream);
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
