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
#ifndef SR_BLOCK_THREADS
#define SR_BLOCK_THREADS 128
#endif
#ifndef SR_MIN_BLOCKS_PER_SM
#define SR_MIN_BLOCKS_PER_SM 5
#endif
constexpr int kBlockThreads = SR_BLOCK_THREADS;
// Launch shape of the fused-step kernels, from a sweep on B200 (6.7B flat buffer): 128-thread
// blocks with at least 5 resident per SM (96 registers per thread, 640 threads per SM) was the
// best of 64..512 threads x 1..10 blocks; tighter register budgets cost more in instruction
// scheduling than they gain in occupancy.
constexpr int kMinBlocksPerSM = SR_MIN_BLOCKS_PER_SM;

struct DeviceInfo {
    int sm_count;
    int cc_major;
};

cudaError_t launch_downcast(const float* src, uint16_t* dst, uint64_t n, uint64_t elem_offset, uint32_t tensor_id,
                            uint32_t seed_hi, const PhiloxKeys& K, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_adamw_flat(uint16_t* p, const void* g, bool g_f32, uint16_t* m, uint16_t* v, uint64_t n,
                              uint64_t elem_offset, uint32_t tensor_id, uint32_t seed_hi, uint32_t flags,
                              const PhiloxKeys& K, const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_adamw_mt(const MtWork* work, uint32_t num_chunks, bool g_f32,
                            uint32_t tensor_id_base, uint32_t seed_hi, uint32_t flags, const PhiloxKeys& K,
                            const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_master_adamw(float* p, uint16_t* p16, const void* g, bool g_f32, float* m, float* v, uint64_t n,
                                const StepScalars& S, const DeviceInfo& dev, cudaStream_t stream);

// Squared norm: number of doubles of scratch needed, and the launcher.
uint64_t sqnorm_scratch_doubles(uint64_t n);
cudaError_t launch_sqnorm(const void* g, bool g_f32, uint64_t n, double* out, double* scratch,
                          const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_clip_scale(const double* sqnorm, float accum_scale, float max_norm, float* out,
                              cudaStream_t stream);

}  // namespace sradamw
