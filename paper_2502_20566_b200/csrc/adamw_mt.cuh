// Multi-tensor kernel of the fused SR-AdamW step and its launcher, for one gradient type.
#pragma once

#include "adamw_body.cuh"

namespace sradamw {

// One work-table entry held in registers.
struct WorkRegs {
    uint16_t* p;
    const void* g;
    uint16_t* m;
    uint16_t* v;
    uint64_t idx0;
    uint32_t len;
    uint32_t tensor_vec;
    __device__ __forceinline__ uint32_t nvec() const { return (tensor_vec >> 31) ? (len >> 3) : 0u; }   // 16-byte vectors
    __device__ __forceinline__ uint32_t tensor() const { return tensor_vec & 0x7FFFFFFFu; }
};

__device__ __forceinline__ WorkRegs load_work(const MtWork* entry) {
    const uint4* q = reinterpret_cast<const uint4*>(entry);
    const uint4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
    WorkRegs w;
    w.p = reinterpret_cast<uint16_t*>(static_cast<uintptr_t>(a.x) | (static_cast<uintptr_t>(a.y) << 32));
    w.g = reinterpret_cast<const void*>(static_cast<uintptr_t>(a.z) | (static_cast<uintptr_t>(a.w) << 32));
    w.m = reinterpret_cast<uint16_t*>(static_cast<uintptr_t>(b.x) | (static_cast<uintptr_t>(b.y) << 32));
    w.v = reinterpret_cast<uint16_t*>(static_cast<uintptr_t>(b.z) | (static_cast<uintptr_t>(b.w) << 32));
    w.idx0 = static_cast<uint64_t>(c.x) | (static_cast<uint64_t>(c.y) << 32);
    w.len = c.z;
    w.tensor_vec = c.w;
    return w;
}

__device__ __forceinline__ WorkRegs no_work() {
    WorkRegs w;
    w.p = nullptr; w.g = nullptr; w.m = nullptr; w.v = nullptr;
    w.idx0 = 0; w.len = 0; w.tensor_vec = 0;
    return w;
}

// Blocks walk the work table (entry c, c + gridDim, ...); the entry after the current one is already
// in registers.  Element indices restart at 0 in every tensor and chunk starts are multiples of 8,
// so an aligned tensor is processed as whole noise groups.  Tensors whose buffers are not 16-byte
// aligned go element by element.
// MODE 1: reference arithmetic; 2 / 3: branch-free arithmetic without / with the gradient scale.
// STAGED (modes 2, 3): every thread keeps its next vector in flight through shared memory with
// asynchronous copies, across chunk boundaries as well: during its last vector of a chunk it
// already fetches its first vector of the next chunk.
template <bool G32, uint32_t FLAGS, int MODE, bool STAGED, bool EPS_IN>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocksPerSM)
k_sr_adamw_mt(const MtWork* __restrict__ work, uint32_t num_chunks, uint32_t tensor_id_base, uint32_t seed_hi,
              const __grid_constant__ PhiloxKeys K, const __grid_constant__ StepScalars S) {
    constexpr int kArrays = G32 ? 5 : 4;
    constexpr bool kStage = STAGED && MODE >= 2;
    constexpr int kVar = (MODE == 3 ? 1 : 0) | (EPS_IN ? 2 : 0);   // bit 0: gradient scale, bit 1: epsilon under the root
    __shared__ uint4 stage[kStage ? kMtStages * kArrays * kBlockThreads : 1];
    static_assert(kMtStages == 2, "slot bookkeeping below assumes two stages");
    const float gscale = S.gscale_dev ? __ldg(S.gscale_dev) : S.gscale;
    const uint32_t tid = threadIdx.x;
    uint4* const mine = stage + tid;
    auto slot = [&](int s, int a) -> uint4* { return mine + (s * kArrays + a) * kBlockThreads; };
    auto issue = [&](const WorkRegs& W, uint32_t j, int s) {   // copies of vector j of chunk W into stage s
        async_copy16(slot(s, 0), reinterpret_cast<const uint4*>(W.p) + j);
        async_copy16(slot(s, 1), reinterpret_cast<const uint4*>(W.m) + j);
        async_copy16(slot(s, 2), reinterpret_cast<const uint4*>(W.v) + j);
        if (G32) {
            async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(W.g) + 2 * j);
            async_copy16(slot(s, 4), reinterpret_cast<const uint4*>(W.g) + 2 * j + 1);
        } else {
            async_copy16(slot(s, 3), reinterpret_cast<const uint4*>(W.g) + j);
        }
    };

    uint32_t c = blockIdx.x;
    WorkRegs cur = c < num_chunks ? load_work(work + c) : no_work();
    WorkRegs nxt = (c < num_chunks && num_chunks - c > gridDim.x) ? load_work(work + c + gridDim.x) : no_work();
    int s = 0;
    if (kStage) {
        if (tid < cur.nvec()) issue(cur, tid, 0);
        async_copy_commit();
    }
    while (c < num_chunks) {
        const uint32_t nvec = cur.nvec(), nvec_next = nxt.nvec();
        const uint32_t c1 = static_cast<uint32_t>(cur.idx0 >> 33);
        const uint32_t c2 = tensor_id_base + cur.tensor();
        if ((cur.tensor_vec >> 31) && MODE >= 2 && !kStage) {
            // direct loads with a register double buffer: my next vector of this chunk is requested before the
            // current one is computed
            uint4 pv = make_uint4(0, 0, 0, 0), mv = pv, vv = pv, g0 = pv, g1 = pv;
            auto load = [&](uint32_t j, uint4& a, uint4& b, uint4& c, uint4& d0, uint4& d1) {
                if (j < nvec) {
                    a = ld16(cur.p, j);
                    b = ld16(cur.m, j);
                    c = ld16(cur.v, j);
                    if (G32) {
                        d0 = ld16(cur.g, 2 * j);
                        d1 = ld16(cur.g, 2 * j + 1);
                    } else {
                        d0 = ld16(cur.g, j);
                    }
                }
            };
            load(tid, pv, mv, vv, g0, g1);
            for (uint32_t j = tid; j < nvec; j += kBlockThreads) {
                uint4 pn = pv, mn = mv, vn = vv, gn0 = g0, gn1 = g1;
                load(j + kBlockThreads, pn, mn, vn, gn0, gn1);
                float ge[8];
                unpack_grad8<G32>(g0, g1, ge);
                step_vec8_fast_loaded<G32, FLAGS, kVar>(cur.p, cur.g, cur.m, cur.v, j, cur.idx0 + (static_cast<uint64_t>(j) << 3), pv,
                                                             mv, vv, ge, c1, c2, seed_hi, gscale, K, S);
                pv = pn; mv = mn; vv = vn; g0 = gn0; g1 = gn1;
            }
            const uint32_t done = nvec << 3;
            if (tid < cur.len - done)
                step_scalar<G32, FLAGS>(cur.p, cur.g, cur.m, cur.v, done + tid, cur.idx0 + done + tid, c2, seed_hi, gscale, K, S);
        } else if (cur.tensor_vec >> 31) {
            for (uint32_t j = tid; j < nvec; j += kBlockThreads) {
                const uint64_t idx0 = cur.idx0 + (static_cast<uint64_t>(j) << 3);
                if (MODE == 1) {
                    step_vec8_reference<G32, FLAGS, true>(cur.p, cur.g, cur.m, cur.v, j, idx0, c2, seed_hi, gscale, K, S);
                } else if (!kStage) {
                    step_vec8_fast<G32, FLAGS, kVar>(cur.p, cur.g, cur.m, cur.v, j, idx0, c1, c2, seed_hi, gscale, K, S);
                } else {
                    // fetch ahead: my next vector of this chunk, else my first vector of the next chunk
                    if (j + kBlockThreads < nvec) issue(cur, j + kBlockThreads, s ^ 1);
                    else if (tid < nvec_next) issue(nxt, tid, s ^ 1);
                    async_copy_commit();
                    async_copy_wait<1>();   // the group holding vector j has landed
                    const uint4 pv = *slot(s, 0), mv = *slot(s, 1), vv = *slot(s, 2);
                    float ge[8];
                    unpack_grad8<G32>(*slot(s, 3), G32 ? *slot(s, kArrays - 1) : make_uint4(0, 0, 0, 0), ge);
                    step_vec8_fast_loaded<G32, FLAGS, kVar>(cur.p, cur.g, cur.m, cur.v, j, idx0, pv, mv, vv, ge, c1, c2,
                                                                 seed_hi, gscale, K, S);
                    s ^= 1;
                }
            }
            if (kStage && tid >= nvec) {   // no vector of mine in this chunk: nothing was fetched ahead yet
                if (tid < nvec_next) issue(nxt, tid, s);
                async_copy_commit();
            }
            const uint32_t done = nvec << 3;
            if (tid < cur.len - done)
                step_scalar<G32, FLAGS>(cur.p, cur.g, cur.m, cur.v, done + tid, cur.idx0 + done + tid, c2, seed_hi, gscale, K, S);
        } else {
            for (uint32_t j = tid; j < cur.len; j += kBlockThreads)
                step_scalar<G32, FLAGS>(cur.p, cur.g, cur.m, cur.v, j, cur.idx0 + j, c2, seed_hi, gscale, K, S);
            if (kStage) {
                if (tid < nvec_next) issue(nxt, tid, s);
                async_copy_commit();
            }
        }
        cur = nxt;
        c += gridDim.x;
        nxt = (c < num_chunks && num_chunks - c > gridDim.x) ? load_work(work + c + gridDim.x) : no_work();
    }
    if (kStage) async_copy_wait<0>();
}

#ifndef SR_STAGE_MT_BF16
#define SR_STAGE_MT_BF16 1
#endif
#ifndef SR_STAGE_MT_F32
#define SR_STAGE_MT_F32 0
#endif

template <bool G32, uint32_t FLAGS, int MODE, bool EPS_IN = false>
cudaError_t launch_mt_mode(const MtWork* work, uint32_t num_chunks, uint32_t tensor_id_base, uint32_t seed_hi,
                           const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr bool kStaged = G32 ? (SR_STAGE_MT_F32 != 0) : (SR_STAGE_MT_BF16 != 0);
    auto k = k_sr_adamw_mt<G32, FLAGS, MODE, kStaged, EPS_IN>;
    const unsigned resident = static_cast<unsigned>(resident_blocks(k, dev));
    const unsigned grid = num_chunks < resident ? num_chunks : resident;
    k<<<grid, kBlockThreads, 0, stream>>>(work, num_chunks, tensor_id_base, seed_hi, K, S);
    return cudaGetLastError();
}

template <bool G32, uint32_t FLAGS>
cudaError_t launch_mt_flags(const MtWork* work, uint32_t num_chunks, uint32_t tensor_id_base, uint32_t seed_hi,
                            const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream) {
    if (!fast_path_allowed(S))
        return launch_mt_mode<G32, FLAGS, 1>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
    if (S.eps_inside)
        return needs_scale(S) ? launch_mt_mode<G32, FLAGS, 3, true>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream)
                              : launch_mt_mode<G32, FLAGS, 2, true>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
    if (needs_scale(S))
        return launch_mt_mode<G32, FLAGS, 3>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
    return launch_mt_mode<G32, FLAGS, 2>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream);
}

template <bool G32>
cudaError_t launch_adamw_mt_g(const MtWork* work, uint32_t num_chunks, uint32_t tensor_id_base, uint32_t seed_hi,
                              uint32_t flags, const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev,
                              cudaStream_t stream) {
#define SR_MT(F) launch_mt_flags<G32, F>(work, num_chunks, tensor_id_base, seed_hi, K, S, dev, stream)
    SR_DISPATCH_FLAGS(SR_MT)
#undef SR_MT
}

}  // namespace sradamw
