// Internal launcher interface between the C-ABI layer (api.cu) and the kernel translation units.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "device_math.cuh"

namespace sradamw {

// Device-side work table of a multi-tensor plan: one entry per chunk (up to kMtChunkElems consecutive
// elements of one tensor) with the four pointers already advanced to the chunk's first element, so a
// block needs a single 48-byte read per chunk and can fetch the next entry while it works.
struct MtWork {
    uint16_t* p;
    const void* g;
    uint16_t* m;
    uint16_t* v;
    uint64_t idx0;        // index of the chunk's first element inside its tensor (multiple of kMtChunkElems)
    uint32_t len;         // elements in this chunk
    uint32_t tensor_vec;  // tensor index (bits 0..30) | bit 31: all four tensor buffers are 16-byte aligned
};
static_assert(sizeof(MtWork) == 48, "three 16-byte loads per entry");

constexpr uint32_t kMtChunkElems = 8192;   // multiple of 8; never crosses a multiple of 2^33
// Launch shapes, from sweeps on B200 with the 6.7B flat buffer (64..512 threads x 1..10 blocks/SM x
// 2..6 stages on the real kernels).  Every kernel's arithmetic needs about 96 registers; tighter
// budgets cost more in instruction scheduling than they gain in occupancy.
//  - kernels that load straight into registers: 128 threads, >= 5 blocks/SM (640 threads/SM);
//  - the staged flat kernel (BF16 gradients): ONE block of 384 threads per SM, 3 vectors per thread in flight or
//    in use (72 KB of dynamic shared memory).  With the memory latency covered by the staging, few resident
//    warps run fastest, at every launch length.  6.7B elements, two GPUs, first 20 launches / 3 s sustained:
//    384 x 1 x 3 stages 15.56-15.60 / 16.13-16.18 ms, 512 x 1 x 2 the same, 256 x 2 x 3 (the shape before)
//    15.84-15.90 / 16.24-16.27, 384 x 1 x 4 15.72-15.76 / 16.14, 512 x 1 x 3 15.84-15.95 / 16.14-16.17,
//    256 x 2 x 4 and x 5 as x 3, 192 x 2 x 3 16.0 / 16.55, 384 x 1 x 2 16.35 / 16.9, 320 x 1 x 3 17.2 / 17.9, 448 x 1 x 3
//    16.7 / 16.7, 256 x 3 x 4 16.8 / 17.5 (the irregular ones: the grid's stride in memory matters as well).
//    Against 128 x 5 x 2 stages, the shape short launches used to take, same GPU: 2^23 elements 0.0205 vs
//    0.0225 ms, 2^26 0.150 vs 0.158, 2^28 0.594 vs 0.628, 355M 0.785 vs 0.834, 832M 1.86 vs 1.96, 2^31 4.87 vs 5.10;
//    equal below 2^22 elements (launch latency);
//  - the staged multi-tensor kernel keeps 128 x 5 with 2 stages.
#ifndef SR_BLOCK_THREADS
#define SR_BLOCK_THREADS 128
#endif
#ifndef SR_MIN_BLOCKS_PER_SM
#define SR_MIN_BLOCKS_PER_SM 5
#endif
#ifndef SR_FLAT_STAGED_THREADS
#define SR_FLAT_STAGED_THREADS 384
#endif
#ifndef SR_FLAT_STAGED_MIN_BLOCKS
#define SR_FLAT_STAGED_MIN_BLOCKS 1
#endif
#ifndef SR_FLAT_STAGES
#define SR_FLAT_STAGES 3
#endif
// the flat step with FP32 gradients, 832M elements, same GPU.  All five 16-byte pieces of a vector loaded into a
// register double buffer: 256 x 2 2.20 ms, 128 x 4 2.21, 128 x 5 2.26, 384 x 1 2.39, 128 x 3 2.40 (bound by load
// latency at 128 registers); all five staged like the BF16 kernel: 2.58-2.60; x, m, v staged and the gradient in the
// register double buffer: 512 x 1 x 2 stages 2.06 ms, 512 x 1 x 3 2.06, 256 x 2 x 3 2.07, 384 x 1 x 3 2.08.  The direct
// shape remains for offsets that are not multiples of 8.
constexpr int kFlatDirectThreads = 256;
constexpr int kFlatDirectMinBlocks = 2;
// A flat call is cut into launches of 2^28 elements (the last one up to 1.5 times that).  Mid-size launches run faster
// per element than one huge one wherever the board is not yet on its power cap: 6.7B elements, first 20 calls /
// sustained, cut at 2^26, 2^27, 2^28, 2^29, not at all: 14.96 / 15.60, 14.85 / 15.45, 14.80 / 15.36, 14.88 / 15.36,
// 15.31 / 15.46 ms on a GPU that sustains 1.67 GHz, and 15.66 / 16.45 (2^28) against 15.78 / 16.43 ms (not cut) on one
// that sustains 1.55 GHz.
constexpr uint64_t kFlatLaunchElems = static_cast<uint64_t>(1) << 28;
// the cut points of a flat call: lengths of its launches in order (shared by the launcher and the launch count)
inline uint64_t next_flat_launch(uint64_t idx, uint64_t left) {
    const uint64_t to_boundary = (static_cast<uint64_t>(1) << 33) - (idx & ((static_cast<uint64_t>(1) << 33) - 1));
    uint64_t len = left < to_boundary ? left : to_boundary;   // every index of a launch has the same index >> 33
    if (len > kFlatLaunchElems + kFlatLaunchElems / 2) len = kFlatLaunchElems;   // a multiple of 8: alignment and noise groups carry over
    return len;
}
constexpr int kFlatStagedThreadsF32 = 512;
constexpr int kFlatStagesF32 = 2;
constexpr int kBlockThreads = SR_BLOCK_THREADS;
constexpr int kMinBlocksPerSM = SR_MIN_BLOCKS_PER_SM;
constexpr int kFlatStagedThreads = SR_FLAT_STAGED_THREADS;
constexpr int kFlatStagedMinBlocks = SR_FLAT_STAGED_MIN_BLOCKS;
constexpr int kFlatStages = SR_FLAT_STAGES;
constexpr int kMtStages = 2;

constexpr int kMaxDevices = 64;
struct DeviceInfo {
    int sm_count;
    int cc_major;
    int index;      // CUDA device ordinal, < kMaxDevices
};

cudaError_t launch_downcast(const float* src, uint16_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                            uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_adamw_flat(uint16_t* p, const void* g, bool g_f32, uint16_t* m, uint16_t* v, uint64_t n,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, uint32_t flags,
                              const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_adamw_mt(const MtWork* work, uint32_t num_chunks, bool g_f32,
                            uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_downcast_fp8(const float* src, uint8_t* dst, uint64_t n, bool e5m2, uint64_t elem_offset,
                                uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev,
                                cudaStream_t stream);

// records e for sr_last_cuda_error() of the calling thread and returns the value of SR_ERR_CUDA
int note_cuda_error(cudaError_t e);
// properties of the current device (cached per device, thread-safe) and, optionally, its index;
// returns an sr_status value
int current_device_info(DeviceInfo* out, int* device_index);

cudaError_t launch_downcast_fp4(const float* src, uint8_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                                uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_accumulate(uint16_t* acc, const void* g, bool g_f32, uint64_t n, float scale, bool stochastic,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, const PhiloxKeys& K,
                              const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_master_adamw(float* p, uint16_t* p16, const void* g, bool g_f32, float* m, float* v, uint64_t n,
                                const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

// mismatches[0 / 1]: square roots / divisions of the branch-free sequences that differ from the IEEE instructions
cudaError_t launch_selftest_in_range(uint64_t sets, uint32_t seed_hi, const PhiloxKeys& K, unsigned long long* mismatches,
                                     const DeviceInfo& dev, cudaStream_t stream);

// Squared norm: number of doubles of scratch needed, and the launcher.
uint64_t sqnorm_scratch_doubles(uint64_t n);
uint64_t sqnorm_mt_scratch_doubles(uint64_t num_chunks);
cudaError_t launch_sqnorm_mt(const MtWork* work, uint32_t num_chunks, bool g_f32, double* out, double* scratch,
                             const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_sqnorm(const void* g, bool g_f32, uint64_t n, double* out, double* scratch,
                          const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_clip_scale(const double* sqnorm, float accum_scale, float max_norm, float* out,
                              cudaStream_t stream);

}  // namespace sradamw
