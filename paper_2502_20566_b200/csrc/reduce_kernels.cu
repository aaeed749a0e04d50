// Squared gradient norm with a fixed FP64 summation tree, and the clipping factor.
//
// The tree is part of the library's contract (the result must not depend on the launch shape):
// blocks of 8192 consecutive entries; inside a block 256 accumulators, accumulator j adding the
// entries r*1024 + 4j + k (r = 0..7, k = 0..3) in that order; 8 warps folded by an XOR butterfly
// (16, 8, 4, 2, 1), warp values added in order 0..7; block sums reduced again by the same rule.
// With FP32 entries a CUDA block of 256 threads is exactly one tree block: thread j is accumulator j and
// its four entries of one r are one 16-byte load.  With BF16 entries four entries are only 8 bytes, so a
// block of 128 threads is one tree block and thread t holds accumulators 2t and 2t + 1, whose eight
// entries of one r are one 16-byte load (same tree, see fold_block_pairs).  HBM-bound: 4 (FP32) or 2
// (BF16) bytes per element.
// Launches per call: one for up to 8192 entries, two for up to 8192^2 (first pass, one block folding the block
// sums), and still two beyond that: the pass over the block sums folds its own results in the block that finishes
// last (k_tree_pass<true>; 355M BF16 entries in a list of 292 tensors: 0.1235 -> 0.1212 ms, and 0.1196 ms with the
// short blocks at tensor ends read as 16-byte vectors too).

#include <atomic>
#include <mutex>

#include "../../include/sradamw.h"
#include "launch.h"

namespace sradamw {

namespace {

constexpr uint32_t kTreeBlock = 8192;
constexpr int kTreeThreads = 256;   // one thread per accumulator of the tree: fixed by the contract

// squares are exact in double for FP32 / BF16 inputs, so fma(g, g, acc) rounds once, exactly like
// acc + g*g
__device__ __forceinline__ double add_square(double acc, float g) {
    const double d = static_cast<double>(g);
    return __fma_rn(d, d, acc);
}

__device__ __forceinline__ double fold_block(double acc, double* warp_sums) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) acc = __dadd_rn(acc, __shfl_xor_sync(0xFFFFFFFFu, acc, s));
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) warp_sums[warp] = acc;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
        total = warp_sums[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) total = __dadd_rn(total, warp_sums[w]);
    }
    __syncthreads();
    return total;   // valid in thread 0
}

// The same tree with two accumulators per thread (thread t: accumulators 2t and 2t + 1, 128 threads).  Tree
// lane l = 2 (t & 15) + b of tree warp t >> 4: the butterfly partners l ^ 16, 8, 4, 2 are the same b in threads
// t ^ 8, 4, 2, 1; the partner l ^ 1 is the thread's other accumulator.  Every addition has the same two
// operands as in fold_block, so the bits are the same.
__device__ __forceinline__ double fold_block_pairs(double a0, double a1, double* warp_sums) {
#pragma unroll
    for (int s = 8; s >= 1; s >>= 1) {
        a0 = __dadd_rn(a0, __shfl_xor_sync(0xFFFFFFFFu, a0, s));
        a1 = __dadd_rn(a1, __shfl_xor_sync(0xFFFFFFFFu, a1, s));
    }
    const double x = __dadd_rn(a0, a1);
    if ((threadIdx.x & 15) == 0) warp_sums[threadIdx.x >> 4] = x;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
        total = warp_sums[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) total = __dadd_rn(total, warp_sums[w]);
    }
    __syncthreads();
    return total;   // valid in thread 0
}

constexpr int kPairThreads = 128;   // BF16 entries: two accumulators per thread
// Resident blocks per SM asked of the compiler for the first passes (their register budgets).  355M entries, same GPU:
// BF16 flat 0.1257 ms with 55 registers (no bound, 9 blocks), 0.1156 with 77 (6 blocks), 0.1132 with 61 (8 blocks);
// BF16 list 0.1196 ms with 80 registers (no bound, 6 blocks), 0.1172 (7), 0.1160 (8), 0.1169 (9 blocks); FP32 list
// 0.2322 ms with 90 registers (no bound, 2 blocks of 256 threads), 0.2090 (3 blocks), 0.2086 (4 blocks).
constexpr int kPairMinBlocks = 8;
constexpr int kListF32MinBlocks = 4;

// One whole, 16-byte aligned tree block of BF16 entries: eight 16-byte loads per thread, all issued before the
// first addition.  t = threadIdx.x of a 128-thread block; returns the block sum in thread 0.
__device__ __forceinline__ double bf16_block_sum(const void* chunk, uint32_t t, double* warp_sums) {
    const uint4* src = reinterpret_cast<const uint4*>(chunk) + t;
    uint4 q[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) q[r] = __ldcs(src + r * 128);
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        a0 = add_square(a0, bf16_lo(q[r].x));
        a0 = add_square(a0, bf16_hi(q[r].x));
        a0 = add_square(a0, bf16_lo(q[r].y));
        a0 = add_square(a0, bf16_hi(q[r].y));
        a1 = add_square(a1, bf16_lo(q[r].z));
        a1 = add_square(a1, bf16_hi(q[r].z));
        a1 = add_square(a1, bf16_lo(q[r].w));
        a1 = add_square(a1, bf16_hi(q[r].w));
    }
    return fold_block_pairs(a0, a1, warp_sums);
}

// A 16-byte aligned tree block of BF16 entries that ends early (`len` < 8192 entries): whole 16-byte vectors inside
// `len` as in bf16_block_sum, the one vector that `len` cuts entry by entry, zeros beyond.  A zero entry adds +0 to
// an accumulator that is never -0, so the bits are those of the rule that skips entries past the end.
__device__ __forceinline__ double bf16_block_sum_short(const uint16_t* chunk, uint32_t len, uint32_t t, double* warp_sums) {
    const uint4* src = reinterpret_cast<const uint4*>(chunk);
    uint4 q[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const uint32_t vec = static_cast<uint32_t>(r) * 128u + t, e0 = 8u * vec;
        q[r] = make_uint4(0u, 0u, 0u, 0u);
        if (e0 + 8u <= len) {
            q[r] = __ldcs(src + vec);
        } else if (e0 < len) {
            uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (uint32_t k = 0; k < 8u; ++k)
                if (e0 + k < len) w[k >> 1] |= static_cast<uint32_t>(chunk[e0 + k]) << (16u * (k & 1u));
            q[r] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        a0 = add_square(a0, bf16_lo(q[r].x));
        a0 = add_square(a0, bf16_hi(q[r].x));
        a0 = add_square(a0, bf16_lo(q[r].y));
        a0 = add_square(a0, bf16_hi(q[r].y));
        a1 = add_square(a1, bf16_lo(q[r].z));
        a1 = add_square(a1, bf16_hi(q[r].z));
        a1 = add_square(a1, bf16_lo(q[r].w));
        a1 = add_square(a1, bf16_hi(q[r].w));
    }
    return fold_block_pairs(a0, a1, warp_sums);
}

// A ragged or unaligned tree block of BF16 entries, `len` of them from `chunk` on: element by element.
__device__ __forceinline__ double bf16_block_sum_ragged(const uint16_t* chunk, uint64_t len, uint32_t t, double* warp_sums) {
    double a[2] = {0.0, 0.0};
    for (int b = 0; b < 2; ++b)
        for (int r = 0; r < 8; ++r)
            for (int k = 0; k < 4; ++k) {
                const uint64_t e = static_cast<uint64_t>(r) * 1024u + 4u * (2u * t + b) + k;
                if (e < len) a[b] = add_square(a[b], __uint_as_float(static_cast<uint32_t>(chunk[e]) << 16));
            }
    return fold_block_pairs(a[0], a[1], warp_sums);
}

// First pass: out[c] = tree-block sum of squares of entries [c*8192, (c+1)*8192) of g.
template <bool G32>
__global__ void __launch_bounds__(G32 ? kTreeThreads : kPairThreads, G32 ? 1 : kPairMinBlocks)
k_sqnorm_pass1(const void* __restrict__ g, uint64_t n, uint64_t num_blocks, bool vec_ok, double* __restrict__ out,
               unsigned long long* ticket) {
    __shared__ double warp_sums[8];
    const uint32_t j = threadIdx.x;
    if (ticket != nullptr && blockIdx.x == 0 && j == 0) *ticket = 0;   // see k_tree_pass<true>
    for (uint64_t c = blockIdx.x; c < num_blocks; c += gridDim.x) {
        const uint64_t base = c * kTreeBlock;
        const bool whole = vec_ok && n - base >= kTreeBlock;
        double total;
        if (!G32) {
            const uint16_t* chunk = static_cast<const uint16_t*>(g) + base;
            total = whole ? bf16_block_sum(chunk, j, warp_sums) : bf16_block_sum_ragged(chunk, n - base, j, warp_sums);
        } else {
            double acc = 0.0;
            if (whole) {
                const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(g) + base) + j;
                float4 q[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) q[r] = __ldcs(src + r * 256);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    acc = add_square(acc, q[r].x);
                    acc = add_square(acc, q[r].y);
                    acc = add_square(acc, q[r].z);
                    acc = add_square(acc, q[r].w);
                }
            } else {
                for (int r = 0; r < 8; ++r)
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t e = base + static_cast<uint64_t>(r) * 1024u + 4u * j + k;
                        if (e < n) acc = add_square(acc, static_cast<const float*>(g)[e]);
                    }
            }
            total = fold_block(acc, warp_sums);
        }
        if (j == 0) out[c] = total;
    }
}

// First pass over a tensor list: out[c] = tree-block sum of squares of work-table entry c (a chunk of
// at most 8192 consecutive gradient entries of one tensor, positions counted from the chunk's start).
template <bool G32>
__global__ void __launch_bounds__(G32 ? kTreeThreads : kPairThreads, G32 ? kListF32MinBlocks : kPairMinBlocks)
k_sqnorm_mt_pass1(const MtWork* __restrict__ work, uint32_t num_chunks, double* __restrict__ out,
                  unsigned long long* ticket) {
    __shared__ double warp_sums[8];
    const uint32_t j = threadIdx.x;
    if (ticket != nullptr && blockIdx.x == 0 && j == 0) *ticket = 0;   // see k_tree_pass<true>
    // the entry after the current one is fetched before the current chunk's data, so that its latency
    // is not paid between chunks
    uint64_t c = blockIdx.x;
    const void* g = nullptr;
    uint32_t len = 0;
    if (c < num_chunks) {
        g = work[c].g;
        len = work[c].len;
    }
    for (; c < num_chunks; c += gridDim.x) {
        const uint64_t cn = c + gridDim.x;
        const void* g_next = nullptr;
        uint32_t len_next = 0;
        if (cn < num_chunks) {
            g_next = work[cn].g;
            len_next = work[cn].len;
        }
        const bool aligned = (reinterpret_cast<uintptr_t>(g) & 15u) == 0;
        const bool whole = len == kTreeBlock && aligned;
        double total;
        if (!G32) {
            total = whole     ? bf16_block_sum(g, j, warp_sums)
                    : aligned ? bf16_block_sum_short(static_cast<const uint16_t*>(g), len, j, warp_sums)
                              : bf16_block_sum_ragged(static_cast<const uint16_t*>(g), len, j, warp_sums);
        } else {
            double acc = 0.0;
            if (whole) {
                const float4* src = reinterpret_cast<const float4*>(g) + j;
                float4 q[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) q[r] = __ldcs(src + r * 256);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    acc = add_square(acc, q[r].x);
                    acc = add_square(acc, q[r].y);
                    acc = add_square(acc, q[r].z);
                    acc = add_square(acc, q[r].w);
                }
            } else {
                for (int r = 0; r < 8; ++r)
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t e = static_cast<uint32_t>(r) * 1024u + 4u * j + k;
                        if (e < len) acc = add_square(acc, static_cast<const float*>(g)[e]);
                    }
            }
            total = fold_block(acc, warp_sums);
        }
        if (j == 0) out[c] = total;
        g = g_next;
        len = len_next;
    }
}

// Later passes: the same rule on an array of doubles (no squaring).  LAST: this pass leaves at most one tree block
// of values (2 <= num_blocks <= 8192) and the block that finishes last folds them into *result, so the final level
// needs no launch of its own.  *result serves as the count of finished blocks until then: the first pass of the call
// has set it to zero.  The additions and their order are those of a separate launch.
template <bool LAST>
__global__ void __launch_bounds__(kTreeThreads)
k_tree_pass(const double* __restrict__ in, uint64_t count, uint64_t num_blocks, double* out, double* result) {
    __shared__ double warp_sums[8];
    __shared__ bool is_last;
    const uint32_t j = threadIdx.x;
    for (uint64_t c = blockIdx.x; c < num_blocks; c += gridDim.x) {
        const uint64_t base = c * kTreeBlock;
        double acc = 0.0;
        for (int r = 0; r < 8; ++r)
            for (int k = 0; k < 4; ++k) {
                const uint64_t e = base + static_cast<uint64_t>(r) * 1024u + 4u * j + k;
                if (e < count) acc = __dadd_rn(acc, in[e]);
            }
        const double total = fold_block(acc, warp_sums);
        if (j == 0) out[c] = total;
    }
    if (!LAST) return;
    if (j == 0) {
        __threadfence();                                          // this block's values before its ticket
        const unsigned t = atomicAdd(reinterpret_cast<unsigned*>(result), 1u);
        is_last = t == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double acc = 0.0;
    for (int r = 0; r < 8; ++r)
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = static_cast<uint32_t>(r) * 1024u + 4u * j + k;
            if (e < num_blocks) acc = __dadd_rn(acc, __ldcg(out + e));   // written by other blocks: read from L2
        }
    const double total = fold_block(acc, warp_sums);
    if (j == 0) *result = total;
}

__global__ void k_clip_scale(const double* __restrict__ sqnorm, float accum_scale, float max_norm,
                             float* __restrict__ out) {
    const double a = static_cast<double>(accum_scale);
    const double norm = __dmul_rn(a, __dsqrt_rn(*sqnorm));
    double coef = __ddiv_rn(static_cast<double>(max_norm), __dadd_rn(norm, 1e-6));
    if (coef > 1.0) coef = 1.0;
    *out = __double2float_rn(__dmul_rn(a, coef));
}

inline uint64_t blocks_of(uint64_t count) { return (count + kTreeBlock - 1) / kTreeBlock; }
// a pass over `count` values that leaves 2 .. 8192 of them also folds those (k_tree_pass<true>)
inline bool merges_last_level(uint64_t count) { return count > kTreeBlock && blocks_of(count) <= kTreeBlock; }

// persistent grid of a first pass: as many blocks as are resident at once
template <typename Kernel>
uint64_t resident_cap(Kernel kernel, int threads, const DeviceInfo& dev) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    return static_cast<uint64_t>(dev.sm_count) * static_cast<uint64_t>(per_sm);
}

// the levels after the first pass: `count` values at level_out (count > 1: inside the scratch), down to *out
cudaError_t launch_tree_levels(double* level_out, uint64_t count, double* out, const DeviceInfo& dev, cudaStream_t stream) {
    const uint64_t cap = static_cast<uint64_t>(dev.sm_count) * 8u;
    while (count > 1) {
        const uint64_t next = blocks_of(count);
        const double* level_in = level_out;
        level_out = next == 1 ? out : level_out + count;
        const unsigned grid = static_cast<unsigned>(next < cap ? next : cap);
        if (merges_last_level(count)) {
            k_tree_pass<true><<<grid, kTreeThreads, 0, stream>>>(level_in, count, next, level_out, out);
            count = 1;
        } else {
            k_tree_pass<false><<<grid, kTreeThreads, 0, stream>>>(level_in, count, next, level_out, nullptr);
            count = next;
        }
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

}  // namespace

// Scratch holds every intermediate level: ceil(n/8192) + ceil(that/8192) + ... down to, but not
// including, the final single value (which goes to the caller's output).
uint64_t sqnorm_scratch_doubles(uint64_t n) {
    uint64_t total = 0;
    uint64_t count = blocks_of(n);
    while (count > 1) {
        total += count;
        count = blocks_of(count);
    }
    return total;
}

// Scratch of the list norm: one double per chunk plus every later level (nothing for 0 or 1 chunks).
uint64_t sqnorm_mt_scratch_doubles(uint64_t num_chunks) {
    uint64_t total = 0;
    uint64_t count = num_chunks;
    while (count > 1) {
        total += count;
        count = blocks_of(count);
    }
    return total;
}

cudaError_t launch_sqnorm_mt(const MtWork* work, uint32_t num_chunks, bool g_f32, double* out, double* scratch,
                             const DeviceInfo& dev, cudaStream_t stream) {
    if (num_chunks == 0) return cudaMemsetAsync(out, 0, sizeof(double), stream);
    uint64_t count = num_chunks;
    double* level_out = count == 1 ? out : scratch;
    // a call with more than one later level counts finished blocks in *out before the result is written there
    unsigned long long* ticket = count > kTreeBlock ? reinterpret_cast<unsigned long long*>(out) : nullptr;
    {
        if (g_f32) {
            const uint64_t res = resident_cap(k_sqnorm_mt_pass1<true>, kTreeThreads, dev);
            k_sqnorm_mt_pass1<true><<<static_cast<unsigned>(count < res ? count : res), kTreeThreads, 0, stream>>>(work, num_chunks, level_out, ticket);
        } else {
            const uint64_t res = resident_cap(k_sqnorm_mt_pass1<false>, kPairThreads, dev);
            k_sqnorm_mt_pass1<false><<<static_cast<unsigned>(count < res ? count : res), kPairThreads, 0, stream>>>(work, num_chunks, level_out, ticket);
        }
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return launch_tree_levels(level_out, count, out, dev, stream);
}

cudaError_t launch_sqnorm(const void* g, bool g_f32, uint64_t n, double* out, double* scratch,
                          const DeviceInfo& dev, cudaStream_t stream) {
    if (n == 0) return cudaMemsetAsync(out, 0, sizeof(double), stream);
    uint64_t count = blocks_of(n);
    double* level_out = count == 1 ? out : scratch;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(g) & 15u) == 0;
    unsigned long long* ticket = count > kTreeBlock ? reinterpret_cast<unsigned long long*>(out) : nullptr;
    {
        if (g_f32) {
            const uint64_t res = resident_cap(k_sqnorm_pass1<true>, kTreeThreads, dev);
            k_sqnorm_pass1<true><<<static_cast<unsigned>(count < res ? count : res), kTreeThreads, 0, stream>>>(g, n, count, vec_ok, level_out, ticket);
        } else {
            const uint64_t res = resident_cap(k_sqnorm_pass1<false>, kPairThreads, dev);
            k_sqnorm_pass1<false><<<static_cast<unsigned>(count < res ? count : res), kPairThreads, 0, stream>>>(g, n, count, vec_ok, level_out, ticket);
        }
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return launch_tree_levels(level_out, count, out, dev, stream);
}

cudaError_t launch_clip_scale(const double* sqnorm, float accum_scale, float max_norm, float* out,
                              cudaStream_t stream) {
    k_clip_scale<<<1, 1, 0, stream>>>(sqnorm, accum_scale, max_norm, out);
    return cudaGetLastError();
}

}  // namespace sradamw

// ---- squared norm without any allocation ---------------------------------------------------
// Same kernels and same summation tree as grad_sqnorm; the intermediate block sums go to a
// fixed array that is part of the library image instead of a caller-provided workspace.

namespace {

constexpr uint64_t kStaticScratchDoubles = 131072;   // 1 MiB per GPU that loads the library

static __device__ __align__(256) double g_sqnorm_static_scratch[kStaticScratchDoubles];

struct StaticScratchSlot {
    std::atomic<bool> ready{false};   // published after ptr
    double* ptr = nullptr;            // device address of g_sqnorm_static_scratch on this device
};
constexpr int kStaticMaxDevices = 64;
StaticScratchSlot g_static_slots[kStaticMaxDevices];
std::mutex g_static_mutex;            // first call on a device: one thread resolves the address, the others wait

}  // namespace

extern "C" uint64_t grad_sqnorm_static_max_elements(void) {
    // largest n whose intermediate levels fit: blocks(n) + blocks(blocks(n)) + ... <= capacity
    uint64_t lo = 0, hi = kStaticScratchDoubles * 8192ull;
    while (lo < hi) {
        const uint64_t mid = lo + (hi - lo + 1) / 2;
        if (sradamw::sqnorm_scratch_doubles(mid) <= kStaticScratchDoubles) lo = mid; else hi = mid - 1;
    }
    return lo;
}

extern "C" sr_status grad_sqnorm_static(const void* g, sr_dtype g_dtype, uint64_t n, double* out_dev, void* stream) {
    if (out_dev == nullptr) return SR_ERR_INVALID_ARG;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (n != 0 && g == nullptr) return SR_ERR_INVALID_ARG;
    if (sradamw::sqnorm_scratch_doubles(n) > kStaticScratchDoubles) return SR_ERR_WORKSPACE;   // n too large
    int dev = 0;
    sradamw::DeviceInfo info;
    const int st = sradamw::current_device_info(&info, &dev);
    if (st != SR_OK) return static_cast<sr_status>(st);
    if (dev < 0 || dev >= kStaticMaxDevices) return SR_ERR_UNSUPPORTED_DEVICE;
    StaticScratchSlot& slot = g_static_slots[dev];
    cudaError_t e;
    if (!slot.ready.load(std::memory_order_acquire)) {
        // once per device, with that device current: the array's name is only a host-side handle,
        // the kernels need its address on this device
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!slot.ready.load(std::memory_order_relaxed)) {
            void* addr = nullptr;
            if ((e = cudaGetSymbolAddress(&addr, g_sqnorm_static_scratch)) != cudaSuccess)
                return static_cast<sr_status>(sradamw::note_cuda_error(e));
            if (addr == nullptr) return static_cast<sr_status>(sradamw::note_cuda_error(cudaErrorInvalidSymbol));
            slot.ptr = static_cast<double*>(addr);
            slot.ready.store(true, std::memory_order_release);
        }
    }
    e = sradamw::launch_sqnorm(g, g_dtype == SR_DT_F32, n, out_dev, slot.ptr, info, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : static_cast<sr_status>(sradamw::note_cuda_error(e));
}
