// Vector and element bodies of the fused SR-AdamW step, shared by the flat and the multi-tensor
// kernels.  One read of x, g, m, v and one write of x, m, v per element; Philox, the FP32 update of
// Algorithm 1 and the dithering add stay in registers.
//
// Each thread moves 8 consecutive elements per iteration with 16-byte loads and stores, so a warp
// touches 512 contiguous bytes per array; all accesses carry the streaming (evict-first) hint
// because every byte is used exactly once.
#pragma once

#include "launch.h"

#ifndef SR_PACKED_F32X2
#define SR_PACKED_F32X2 1
#endif

namespace sradamw {

// ---- 16-byte streaming accesses ------------------------------------------------------------
__device__ __forceinline__ uint4 ld16(const void* base, uint64_t vec) {
    return __ldcs(reinterpret_cast<const uint4*>(base) + vec);
}
__device__ __forceinline__ void st16(void* base, uint64_t vec, uint4 val) {
    __stcs(reinterpret_cast<uint4*>(base) + vec, val);
}

// 32-byte accesses (the 256-bit vector loads/stores of sm_100): eight consecutive 32-bit words per
// thread.  A warp then touches each 32-byte sector of its 1 KB once, where two 16-byte accesses at a
// 32-byte stride touch every sector twice.  The address (base + 32 * vec) must be 32-byte aligned.
struct Words8 {
    uint32_t w[8];
};
__device__ __forceinline__ Words8 ld32(const void* base, uint64_t vec) {
    Words8 r;
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]), "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                 : "l"(static_cast<const char*>(base) + 32 * vec));
    return r;
}
__device__ __forceinline__ void st32(void* base, uint64_t vec, const Words8& r) {
    asm volatile("st.global.cs.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 :
                 : "r"(r.w[0]), "r"(r.w[1]), "r"(r.w[2]), "r"(r.w[3]), "r"(r.w[4]), "r"(r.w[5]), "r"(r.w[6]), "r"(r.w[7]),
                   "l"(static_cast<char*>(base) + 32 * vec)
                 : "memory");
}

// ---- asynchronous global -> shared copies (16 bytes, L2 only) ---------------------------------
// Used to keep a thread's NEXT vector in flight while it computes the current one without
// spending registers on it.  Each thread copies into and reads from its own shared-memory slots,
// so no block-level synchronisation is involved; completion is tracked per thread by the
// hardware's copy groups (commit / wait), not by polling.
__device__ __forceinline__ void async_copy16(uint4* smem_dst, const void* gmem_src) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void async_copy_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// returns once at most PENDING of this thread's committed groups are still in flight
template <int PENDING>
__device__ __forceinline__ void async_copy_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// unpack a staged gradient vector (one 16-byte piece for BF16, two for FP32)
template <bool G32>
__device__ __forceinline__ void unpack_grad8(const uint4 g0, const uint4 g1, float (&ge)[8]) {
    if (G32) {
        ge[0] = __uint_as_float(g0.x); ge[1] = __uint_as_float(g0.y);
        ge[2] = __uint_as_float(g0.z); ge[3] = __uint_as_float(g0.w);
        ge[4] = __uint_as_float(g1.x); ge[5] = __uint_as_float(g1.y);
        ge[6] = __uint_as_float(g1.z); ge[7] = __uint_as_float(g1.w);
    } else {
        ge[0] = bf16_lo(g0.x); ge[1] = bf16_hi(g0.x);
        ge[2] = bf16_lo(g0.y); ge[3] = bf16_hi(g0.y);
        ge[4] = bf16_lo(g0.z); ge[5] = bf16_hi(g0.z);
        ge[6] = bf16_lo(g0.w); ge[7] = bf16_hi(g0.w);
    }
}

// the eight gradient values of a vector as FP32
// wide (FP32 gradients only): the gradient buffer is 32-byte aligned, one 32-byte load.  Used by the
// FP32-master kernel; in the SR step kernels it measured 1.8 % slower than the two 16-byte loads
// (same GPU, 832M elements), so they do not ask for it.
template <bool G32>
__device__ __forceinline__ void load_grad8(const void* g, uint64_t vec, float (&ge)[8], bool wide = false) {
    if (G32 && wide) {
        const Words8 r = ld32(g, vec);
#pragma unroll
        for (int e = 0; e < 8; ++e) ge[e] = __uint_as_float(r.w[e]);
    } else if (G32) {
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
}

__device__ __forceinline__ uint32_t word_of(const uint4& w, int j) { return j == 0 ? w.x : j == 1 ? w.y : j == 2 ? w.z : w.w; }

// Noise words of one slot for a vector whose first element sits at position r = idx0 & 7 of its
// noise group: the vector takes the last 8 - r halfwords of group A = idx0 >> 3 and the first r of
// group A + 1, i.e. 128 bits starting at bit 16 r of the 256-bit string (call A : call A + 1).
// r is the same for every vector of a launch, so the word shifts below are uniform selects.
__device__ __forceinline__ uint4 straddling_noise(uint64_t idx0, uint32_t slot, uint32_t c2, uint32_t c3, const PhiloxKeys& K) {
    const uint64_t num_a = ((idx0 >> 3) << 2) | slot, num_b = num_a + 4;
    const uint4 a = philox4x32_10(static_cast<uint32_t>(num_a), static_cast<uint32_t>(num_a >> 32), c2, c3, K);
    const uint4 b = philox4x32_10(static_cast<uint32_t>(num_b), static_cast<uint32_t>(num_b >> 32), c2, c3, K);
    const uint32_t r = static_cast<uint32_t>(idx0) & 7u;
    const bool by2 = (r & 4u) != 0, by1 = (r & 2u) != 0;
    // words r>>1 .. (r>>1)+4 of (a.x a.y a.z a.w b.x b.y b.z b.w)
    const uint32_t x0 = by2 ? a.z : a.x, x1 = by2 ? a.w : a.y, x2 = by2 ? b.x : a.z, x3 = by2 ? b.y : a.w;
    const uint32_t x4 = by2 ? b.z : b.x, x5 = by2 ? b.w : b.y;
    const uint32_t y0 = by1 ? x1 : x0, y1 = by1 ? x2 : x1, y2 = by1 ? x3 : x2, y3 = by1 ? x4 : x3, y4 = by1 ? x5 : x4;
    const uint32_t sh = (r & 1u) * 16u;
    return make_uint4(__funnelshift_r(y0, y1, sh), __funnelshift_r(y1, y2, sh), __funnelshift_r(y2, y3, sh),
                      __funnelshift_r(y3, y4, sh));
}

// The same 128 bits without computing any call twice.  The lanes of a warp hold 32 consecutive vectors (a ROW);
// every lane computes the call of the group its vector ENDS in (group A + 1).  The group its vector starts in is
// the one the previous vector ends in: lanes 1..31 take those words from the lane below by shuffle.  Lane 0 has
// no lane below it: the call of the group its row starts in (the row's HEAD call) comes from a table in shared
// memory that the warp refills every 32 iterations, lane j computing the head call of the row the warp will be
// on j iterations later.  Per (vector, slot) this is 1 + 1/32 calls, against two when every thread computes both
// groups, and the warps keep the plain grid-stride order over rows (whole 512-byte rows, consecutive warps on
// consecutive rows).  R = idx0 & 7 (1..7) is the same for every vector of a launch: the kernels switch on it
// once per vector, so that the word selection is fixed at compile time inside each case.
template <int R>
__device__ __forceinline__ uint4 straddle_select(const uint4 a, const uint4 b) {
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    constexpr int k = R >> 1;
    if (R & 1)   // half a word further: (w[i] >> 16) | (w[i + 1] << 16)
        return make_uint4(__byte_perm(w[k], w[k + 1], 0x5432), __byte_perm(w[k + 1], w[k + 2], 0x5432),
                          __byte_perm(w[k + 2], w[k + 3], 0x5432), __byte_perm(w[k + 3], w[(k + 4) & 7], 0x5432));
    return make_uint4(w[k], w[k + 1], w[k + 2], w[k + 3]);
}

// own: this lane's call (the group its vector ends in); head: where the row's head call lies in shared memory.
// Lanes 1..31 take the words of the lane below; lane 0 loads the head call over them (one predicated 16-byte
// load instead of a select per word: 832M-element step 2.11 -> 2.08 ms, accumulation 0.86 -> 0.84 ms).
// Every lane of the warp must call this (full-mask shuffles).
template <int R>
__device__ __forceinline__ uint4 chain_words(const uint4 own, const uint4* head, uint32_t lane) {
    constexpr int k = R >> 1;   // first word of the starting group that the vector uses
    uint4 a = make_uint4(0, 0, 0, 0);
    if (k <= 0) a.x = __shfl_up_sync(0xFFFFFFFFu, own.x, 1);
    if (k <= 1) a.y = __shfl_up_sync(0xFFFFFFFFu, own.y, 1);
    if (k <= 2) a.z = __shfl_up_sync(0xFFFFFFFFu, own.z, 1);
    a.w = __shfl_up_sync(0xFFFFFFFFu, own.w, 1);
    const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(head));
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %4, 0;\n\t@p ld.shared.v4.u32 {%0, %1, %2, %3}, [%5];\n\t}"
                 : "+r"(a.x), "+r"(a.y), "+r"(a.z), "+r"(a.w)
                 : "r"(lane), "r"(addr)
                 : "memory");
    return straddle_select<R>(a, own);
}

// Noise of a grid-stride walk over rows whose vectors straddle two noise groups.  SLOTS: bit s set = rounding
// slot s is drawn.  FIXED_C1: every index of the launch has the same high counter word c1 (the flat step
// launches are cut that way); otherwise it is taken from the 64-bit call number.  `heads` is this warp's part of
// a shared-memory table: 32 entries of 16 bytes per drawn slot.
template <uint32_t SLOTS, bool FIXED_C1>
struct RowChain {
    static constexpr int kSlots = ((SLOTS >> 0) & 1) + ((SLOTS >> 1) & 1) + ((SLOTS >> 2) & 1) + ((SLOTS >> 3) & 1);
    static constexpr int kTableEntries = 32 * (kSlots > 0 ? kSlots : 1);      // uint4 entries per warp
    static __device__ __forceinline__ int pos(uint32_t s) { return __popc(SLOTS & ((1u << s) - 1u)); }

    uint4* heads;
    uint64_t group0;     // noise group of the launch's first element
    uint64_t stride;     // vectors between a warp's consecutive rows
    uint32_t r, lane, c1, c2, c3;

    // Head calls of the rows this warp is on in iterations k .. k + 31; row_vec0: first vector of its row in
    // iteration k.  Every lane must call it (when k is a multiple of 32, before `words`).
    __device__ __forceinline__ void refill(uint64_t row_vec0, const PhiloxKeys& K) const {
        const uint64_t number = (group0 + row_vec0 + lane * stride) << 2;
        const uint32_t h0 = static_cast<uint32_t>(number), h1 = FIXED_C1 ? c1 : static_cast<uint32_t>(number >> 32);
        __syncwarp();                                                       // the previous 32 entries have been read
#pragma unroll
        for (uint32_t s = 0; s < 4; ++s)
            if (SLOTS & (1u << s)) heads[pos(s) * 32 + lane] = philox4x32_10(h0 | s, h1, c2, c3, K);
        __syncwarp();
    }

    // Noise words w[s] of this lane's vector `vec` in iteration k.  Every lane must call it.
    __device__ __forceinline__ void words(uint64_t vec, uint32_t k, const PhiloxKeys& K, uint4 (&w)[4]) const {
        const uint64_t number = (group0 + vec + 1) << 2;
        const uint32_t c0 = static_cast<uint32_t>(number), c1v = FIXED_C1 ? c1 : static_cast<uint32_t>(number >> 32);
        uint4 own[4];
        const uint4* head[4];
#pragma unroll
        for (uint32_t s = 0; s < 4; ++s)
            if (SLOTS & (1u << s)) {
                own[s] = philox4x32_10(c0 | s, c1v, c2, c3, K);
                head[s] = heads + pos(s) * 32 + (k & 31u);
            }
#define SR_CHAIN_CASE(R)                                                            \
    case R:                                                                         \
        _Pragma("unroll") for (uint32_t s = 0; s < 4; ++s)                          \
            if (SLOTS & (1u << s)) w[s] = chain_words<R>(own[s], head[s], lane);    \
        break;
        switch (r) {
            SR_CHAIN_CASE(1) SR_CHAIN_CASE(2) SR_CHAIN_CASE(3) SR_CHAIN_CASE(4)
            SR_CHAIN_CASE(5) SR_CHAIN_CASE(6) SR_CHAIN_CASE(7)
            default: break;
        }
#undef SR_CHAIN_CASE
    }
};

// ---- reference vector: IEEE square root / division, NaN rule -------------------------------
// GROUPED = true needs idx0 (global index of the vector's first element) to be a multiple of 8: the
// vector is then exactly one noise group and three Philox calls serve it.  GROUPED = false is valid
// for any idx0: the vector straddles two groups and takes six calls.  Kept out of line: the fast
// kernels call it only for the rare vector that leaves the fast range.
template <bool G32, uint32_t FLAGS, bool GROUPED>
__device__ __noinline__ void step_vec8_reference(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t vec,
                                                 uint64_t idx0, uint32_t c2, uint32_t c3, float gscale,
                                                 const PhiloxKeys& K, const StepScalars& S) {
    const uint4 pv = ld16(p, vec), mv = ld16(m, vec), vv = ld16(v, vec);
    float ge[8];
    load_grad8<G32>(g, vec, ge);
    uint4 wx = make_uint4(0, 0, 0, 0), wm = wx, wv = wx;
    if (GROUPED) {
        const uint32_t c0 = static_cast<uint32_t>(idx0 >> 1), c1 = static_cast<uint32_t>(idx0 >> 33);
        if (FLAGS & 1u) wx = philox4x32_10(c0, c1, c2, c3, K);
        if (FLAGS & 2u) wm = philox4x32_10(c0 + 1, c1, c2, c3, K);
        if (FLAGS & 4u) wv = philox4x32_10(c0 + 2, c1, c2, c3, K);
    } else {
        if (FLAGS & 1u) wx = straddling_noise(idx0, 0, c2, c3, K);
        if (FLAGS & 2u) wm = straddling_noise(idx0, 1, c2, c3, K);
        if (FLAGS & 4u) wv = straddling_noise(idx0, 2, c2, c3, K);
    }
    uint32_t po[4], mo[4], vo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t pw = word_of(pv, j), mw = word_of(mv, j), vw = word_of(vv, j);
        const ElementOut r0 = adamw_element(bf16_lo(pw), ge[2 * j], bf16_lo(mw), bf16_lo(vw), gscale, S);
        const ElementOut r1 = adamw_element(bf16_hi(pw), ge[2 * j + 1], bf16_hi(mw), bf16_hi(vw), gscale, S);
        // 16-bit noise per element and slot: the pair's word holds the even element's in its low half
        const uint32_t ax = word_of(wx, j), am = word_of(wm, j), av = word_of(wv, j);
        const uint32_t x0 = ax & 0xFFFFu, x1 = ax >> 16, m0 = am & 0xFFFFu, m1 = am >> 16, v0 = av & 0xFFFFu, v1 = av >> 16;
        po[j] = pack_top_halves(round_sum_r16_nan_safe<(FLAGS & 1u) != 0>(r0.x, x0),
                                round_sum_r16_nan_safe<(FLAGS & 1u) != 0>(r1.x, x1));
        mo[j] = pack_top_halves(round_sum_r16_nan_safe<(FLAGS & 2u) != 0>(r0.m, m0),
                                round_sum_r16_nan_safe<(FLAGS & 2u) != 0>(r1.m, m1));
        vo[j] = pack_top_halves(round_sum_r16_nan_safe<(FLAGS & 4u) != 0>(r0.v, v0),
                                round_sum_r16_nan_safe<(FLAGS & 4u) != 0>(r1.v, v1));
    }
    st16(p, vec, make_uint4(po[0], po[1], po[2], po[3]));
    st16(m, vec, make_uint4(mo[0], mo[1], mo[2], mo[3]));
    st16(v, vec, make_uint4(vo[0], vo[1], vo[2], vo[3]));
}

// ---- fast vector: branch-free arithmetic, one range test per vector ------------------------
// VAR: bit 0 gradient scale, bit 1 epsilon under the square root (see adamw_element_in_range), bit 2: idx0 is not
// a multiple of 8 (only tells the fallback which noise rule applies)
// the vector's noise words (wx, wm, wv: one 16-bit half per element and slot) are given
template <bool G32, uint32_t FLAGS, int VAR>
__device__ __forceinline__ void step_vec8_fast_noise(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t vec,
                                                     uint64_t idx0, const uint4 pv, const uint4 mv, const uint4 vv,
                                                     const float (&ge)[8], const uint4 wx, const uint4 wm, const uint4 wv,
                                                     uint32_t c2, uint32_t c3, float gscale, const PhiloxKeys& K,
                                                     const StepScalars& S) {
    RangeTrack track;
    track.init();
    uint32_t po[4], mo[4], vo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t pw = word_of(pv, j), mw = word_of(mv, j), vw = word_of(vv, j);
#if SR_PACKED_F32X2
        ElementOut r0, r1;
        adamw_pair_in_range<VAR>(bf16_lo(pw), bf16_hi(pw), ge[2 * j], ge[2 * j + 1], bf16_lo(mw), bf16_hi(mw), bf16_lo(vw),
                                   bf16_hi(vw), gscale, S, r0, r1);
#else
        const ElementOut r0 = adamw_element_in_range<VAR>(bf16_lo(pw), ge[2 * j], bf16_lo(mw), bf16_lo(vw), gscale, S);
        const ElementOut r1 = adamw_element_in_range<VAR>(bf16_hi(pw), ge[2 * j + 1], bf16_hi(mw), bf16_hi(vw), gscale, S);
#endif
        track.add(r0, r1);
        po[j] = pack_top_halves(round_sum_word<(FLAGS & 1u) != 0, false>(r0.x, word_of(wx, j)),
                                round_sum_word<(FLAGS & 1u) != 0, true>(r1.x, word_of(wx, j)));
        mo[j] = pack_top_halves(round_sum_word<(FLAGS & 2u) != 0, false>(r0.m, word_of(wm, j)),
                                round_sum_word<(FLAGS & 2u) != 0, true>(r1.m, word_of(wm, j)));
        vo[j] = pack_top_halves(round_sum_word<(FLAGS & 4u) != 0, false>(r0.v, word_of(wv, j)),
                                round_sum_word<(FLAGS & 4u) != 0, true>(r1.v, word_of(wv, j)));
    }
    if (track.left_range()) {
        if (track.zero_vector(S.zero_t_ok)) {
            // all m1 are +-0: u = m1 / den is +-0 with the sign of m1, which the rounded m keeps; only x is redone
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t pw = word_of(pv, j);
                const float x0 = bf16_lo(pw), x1 = bf16_hi(pw);
                const float q0 = __fmaf_rn(S.step_size, bf16_lo(mo[j]), __fmul_rn(S.lr_wd, x0));
                const float q1 = __fmaf_rn(S.step_size, bf16_hi(mo[j]), __fmul_rn(S.lr_wd, x1));
                po[j] = pack_top_halves(round_sum_word_nan_safe<(FLAGS & 1u) != 0, false>(__fsub_rn(x0, q0), word_of(wx, j)),
                                        round_sum_word_nan_safe<(FLAGS & 1u) != 0, true>(__fsub_rn(x1, q1), word_of(wx, j)));
            }
        } else {
            // nothing has been stored yet: redo this vector from memory with the reference arithmetic
            step_vec8_reference<G32, FLAGS, (VAR & 4) == 0>(p, g, m, v, vec, idx0, c2, c3, gscale, K, S);
            return;
        }
    }
    st16(p, vec, make_uint4(po[0], po[1], po[2], po[3]));
    st16(m, vec, make_uint4(mo[0], mo[1], mo[2], mo[3]));
    st16(v, vec, make_uint4(vo[0], vo[1], vo[2], vo[3]));
}

// a vector that is exactly one noise group (idx0 a multiple of 8): three Philox calls, then the above
template <bool G32, uint32_t FLAGS, int VAR>
__device__ __forceinline__ void step_vec8_fast_loaded(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t vec,
                                                      uint64_t idx0, const uint4 pv, const uint4 mv, const uint4 vv,
                                                      const float (&ge)[8], uint32_t c1, uint32_t c2, uint32_t c3,
                                                      float gscale, const PhiloxKeys& K, const StepScalars& S) {
    static_assert((VAR & 4) == 0, "vectors that straddle two noise groups get their words from the caller");
    uint4 wx = make_uint4(0, 0, 0, 0), wm = wx, wv = wx;
    const uint32_t c0 = static_cast<uint32_t>(idx0 >> 1);
    if (FLAGS & 1u) wx = philox4x32_10(c0, c1, c2, c3, K);
    if (FLAGS & 2u) wm = philox4x32_10(c0 + 1, c1, c2, c3, K);
    if (FLAGS & 4u) wv = philox4x32_10(c0 + 2, c1, c2, c3, K);
    step_vec8_fast_noise<G32, FLAGS, VAR>(p, g, m, v, vec, idx0, pv, mv, vv, ge, wx, wm, wv, c2, c3, gscale, K, S);
}

// the same, loading the vector straight into registers
template <bool G32, uint32_t FLAGS, int VAR>
__device__ __forceinline__ void step_vec8_fast(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t vec,
                                               uint64_t idx0, uint32_t c1, uint32_t c2, uint32_t c3, float gscale,
                                               const PhiloxKeys& K, const StepScalars& S) {
    const uint4 pv = ld16(p, vec), mv = ld16(m, vec), vv = ld16(v, vec);
    float ge[8];
    load_grad8<G32>(g, vec, ge);
    step_vec8_fast_loaded<G32, FLAGS, VAR>(p, g, m, v, vec, idx0, pv, mv, vv, ge, c1, c2, c3, gscale, K, S);
}

// ---- one element with 2-byte accesses: ragged tails, unaligned buffers ---------------------
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
    const uint32_t rx = (FLAGS & 1u) ? noise_of_element(idx, 0, c2, c3, K) : 0u;
    const uint32_t rm = (FLAGS & 2u) ? noise_of_element(idx, 1, c2, c3, K) : 0u;
    const uint32_t rv = (FLAGS & 4u) ? noise_of_element(idx, 2, c2, c3, K) : 0u;
    p[i] = static_cast<uint16_t>(round_sum_r16_nan_safe<(FLAGS & 1u) != 0>(r.x, rx) >> 16);
    m[i] = static_cast<uint16_t>(round_sum_r16_nan_safe<(FLAGS & 2u) != 0>(r.m, rm) >> 16);
    v[i] = static_cast<uint16_t>(round_sum_r16_nan_safe<(FLAGS & 4u) != 0>(r.v, rv) >> 16);
}

// ---- launch helpers ------------------------------------------------------------------------
inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

template <typename Kernel>
int resident_blocks(Kernel kernel, const DeviceInfo& dev, int threads = kBlockThreads, size_t dynamic_smem = 0) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, dynamic_smem) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    return per_sm * dev.sm_count;
}

// grid for `work_items` thread-items: no more blocks than are resident at once, no more than needed
template <typename Kernel>
unsigned grid_for(Kernel kernel, uint64_t work_items, const DeviceInfo& dev, int threads = kBlockThreads,
                  size_t dynamic_smem = 0) {
    const uint64_t needed = (work_items + threads - 1) / threads;
    const uint64_t resident = static_cast<uint64_t>(resident_blocks(kernel, dev, threads, dynamic_smem));
    const uint64_t g = needed < resident ? needed : resident;
    return static_cast<unsigned>(g < 1 ? 1 : g);
}

// The branch-free path needs den = sqrt(v1) * rsqrt_bc2 + eps to stay inside the range its
// division was validated for.  With epsilon under the root den = sqrt(t) and the per-vector range test
// on t (<= 2^60) already keeps it there; the bounds on the scalars are kept for both.
inline bool fast_path_allowed(const StepScalars& S) {
    return S.rsqrt_bc2 >= 1.0f && S.rsqrt_bc2 <= 1024.0f && S.eps >= 0.0f && S.eps <= 1.0f;
}
inline bool needs_scale(const StepScalars& S) { return S.gscale_dev != nullptr || S.gscale != 1.0f; }

#define SR_DISPATCH_FLAGS(CALL)                    \
    switch (flags & 7u) {                          \
        case 0: return CALL(0);                    \
        case 1: return CALL(1);                    \
        case 2: return CALL(2);                    \
        case 3: return CALL(3);                    \
        case 4: return CALL(4);                    \
        case 5: return CALL(5);                    \
        case 6: return CALL(6);                    \
        default: return CALL(7);                   \
    }

// per gradient type, defined in adamw_flat_*.cu / adamw_mt_*.cu
template <bool G32>
cudaError_t launch_adamw_flat_g(uint16_t* p, const void* g, uint16_t* m, uint16_t* v, uint64_t n, uint64_t elem_offset,
                                uint32_t tensor_id, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                                const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);
template <bool G32>
cudaError_t launch_adamw_mt_g(const MtWork* work, uint32_t num_chunks,
                              uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                              const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

}  // namespace sradamw
