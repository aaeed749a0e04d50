// C-ABI layer of libsradamw.so: argument checks, per-iteration scalars (Algorithm 1, the m-hat and
// v-hat steps), Philox round keys, multi-tensor plans; all device work is in the kernel files.

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/sradamw.h"
#include "launch.h"

using namespace sradamw;

namespace {

thread_local int tl_last_cuda_error = 0;

sr_status cuda_fail(cudaError_t e) {
    tl_last_cuda_error = static_cast<int>(e);
    return SR_ERR_CUDA;
}

struct DeviceSlot {
    std::atomic<bool> known{false};
    DeviceInfo info{};
};
DeviceSlot g_devices[kMaxDevices];

std::mutex g_device_mutex;   // first query of a device: one thread fills the slot, the others wait

// Properties of the current device, queried once per device (a failed query is retried by the next call).
sr_status current_device(DeviceInfo* out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return SR_ERR_UNSUPPORTED_DEVICE;
    DeviceSlot& slot = g_devices[dev];
    if (!slot.known.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_device_mutex);
        if (!slot.known.load(std::memory_order_relaxed)) {
            int sm = 0, major = 0;
            e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return cuda_fail(e);
            e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
            if (e != cudaSuccess) return cuda_fail(e);
            slot.info.sm_count = sm;
            slot.info.cc_major = major;
            slot.info.index = dev;
            slot.known.store(true, std::memory_order_release);
        }
    }
    if (slot.info.cc_major != 10) return SR_ERR_UNSUPPORTED_DEVICE;
    *out = slot.info;
    return SR_OK;
}

PhiloxKeys make_keys(uint64_t seed, uint32_t step) {
    PhiloxKeys K;
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = step;
    for (int r = 0; r < 10; ++r) {
        K.k0[r] = k0;
        K.k1[r] = k1;
        k0 += kPhiloxW0;
        k1 += kPhiloxW1;
    }
    return K;
}

// beta^t by square-and-multiply in double (no libm: identical bits on every host)
double power_u32(double base, uint32_t e) {
    double r = 1.0;
    while (e) {
        if (e & 1u) r *= base;
        base *= base;
        e >>= 1;
    }
    return r;
}

bool finite_f(float x) { return std::isfinite(x); }

sr_status make_scalars(const sr_adamw_hparams* hp, uint32_t step, StepScalars* S) {
    if (hp == nullptr || hp->struct_size != sizeof(sr_adamw_hparams)) return SR_ERR_INVALID_ARG;
    if (step == 0) return SR_ERR_INVALID_ARG;   // 1 - beta^0 = 0
    if (!finite_f(hp->lr) || hp->lr < 0.0f) return SR_ERR_INVALID_ARG;
    if (!(hp->beta1 >= 0.0f && hp->beta1 < 1.0f) || !(hp->beta2 >= 0.0f && hp->beta2 < 1.0f)) return SR_ERR_INVALID_ARG;
    if (!finite_f(hp->eps) || hp->eps < 0.0f || !finite_f(hp->weight_decay)) return SR_ERR_INVALID_ARG;
    if (hp->grad_scale_dev == nullptr && !finite_f(hp->grad_scale)) return SR_ERR_INVALID_ARG;
    if (hp->flags & ~(7u | SR_FLAG_EPS_INSIDE)) return SR_ERR_INVALID_ARG;
    const double b1 = hp->beta1, b2 = hp->beta2, lr = hp->lr, wd = hp->weight_decay;
    const double bc1 = 1.0 - power_u32(b1, step);
    const double bc2 = 1.0 - power_u32(b2, step);
    S->beta1 = hp->beta1;
    S->beta2 = hp->beta2;
    S->omb1 = 1.0f - hp->beta1;
    S->omb2 = 1.0f - hp->beta2;
    S->step_size = static_cast<float>(lr / bc1);
    S->rsqrt_bc2 = static_cast<float>(1.0 / std::sqrt(bc2));
    S->eps = hp->eps;
    S->lr_wd = static_cast<float>(lr * wd);
    S->gscale = hp->grad_scale;
    S->gscale_dev = hp->grad_scale_dev;
    S->eps_inside = (hp->flags & SR_FLAG_EPS_INSIDE) ? 1u : 0u;
    if (S->eps_inside) {
        S->pre_mul = static_cast<float>(1.0 / bc2);
        S->pre_add = hp->eps;
        S->post_mul = 1.0f;
        S->post_add = 0.0f;
    } else {
        S->pre_mul = 1.0f;
        S->pre_add = 0.0f;
        S->post_mul = S->rsqrt_bc2;
        S->post_add = hp->eps;
    }
    // a zero argument of the square root leaves den = eps: inside the branch-free division's range from 2^-30 on
    S->zero_t_ok = (!S->eps_inside && hp->eps >= 9.313225746154785e-10f) ? 1u : 0u;
    return SR_OK;
}

}  // namespace

namespace sradamw {
int note_cuda_error(cudaError_t e) { return static_cast<int>(cuda_fail(e)); }
int current_device_info(DeviceInfo* out, int* device_index) {
    const sr_status st = current_device(out);
    if (st == SR_OK && device_index != nullptr && cudaGetDevice(device_index) != cudaSuccess) return SR_ERR_CUDA;
    return static_cast<int>(st);
}
}  // namespace sradamw

// A tensor of a list that is stepped by a flat launch of its own (see sr_adamw_multi_tensor).
struct LargeTensor {
    uint16_t* p;
    const void* g;
    uint16_t* m;
    uint16_t* v;
    uint64_t numel;
    uint32_t index;
};
// Tensors of at least this many elements whose four buffers are 16-byte aligned: from here on one flat launch per
// tensor is faster than the tensor's share of the list kernel (B200: flat launches of 2^24 / 2^25 / 2^26 elements run
// at 89 / 91 / 96 % of the copy peak, the list kernel at 84-88 %).
constexpr uint64_t kMtFlatElems = static_cast<uint64_t>(1) << 24;

struct sr_mt_plan {
    MtWork* d_work = nullptr;        // every chunk of every tensor, in list order (the list norm reads this one)
    MtWork* d_small = nullptr;       // the chunks of the tensors that the list kernel steps (inside d_work's allocation)
    uint32_t num_small = 0;
    std::vector<LargeTensor> large;  // the tensors stepped by flat launches
    uint32_t num_tensors = 0;
    uint32_t num_chunks = 0;
    uint64_t total_elements = 0;
    bool g_f32 = false;
    int device = 0;
    // Two or more flat launches alternate between the caller's stream and this one, so that the last blocks of one
    // launch run beside the first blocks of the next (the tensors are disjoint); fork / join by these events.
    cudaStream_t side = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};

static cudaError_t release_plan(sr_mt_plan* plan) {
    if (plan->join) cudaEventDestroy(plan->join);
    if (plan->fork) cudaEventDestroy(plan->fork);
    if (plan->side) cudaStreamDestroy(plan->side);     // returns at once; the stream's work completes first
    const cudaError_t e = cudaFree(plan->d_work);
    delete plan;
    return e;
}

extern "C" {

sr_status sr_downcast_f32_bf16(const float* src, uint16_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                               uint32_t tensor_id, uint64_t elem_offset, void* stream) {
    if (n == 0) return SR_OK;
    if (src == nullptr || dst == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_downcast(src, dst, n, elem_offset, tensor_id, static_cast<uint32_t>(seed >> 32),
                                          make_keys(seed, step), dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

uint32_t sr_adamw_step_launch_count(uint64_t n, uint64_t elem_offset) {
    uint32_t count = 0;
    for (uint64_t done = 0; done < n; ++count) done += next_flat_launch(elem_offset + done, n - done);
    return count;
}

sr_status sr_selftest_in_range_arithmetic(uint64_t seed, uint64_t sets, uint64_t* mismatches_dev, void* stream) {
    if (mismatches_dev == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_selftest_in_range(sets, static_cast<uint32_t>(seed >> 32), make_keys(seed, 0),
                                                   reinterpret_cast<unsigned long long*>(mismatches_dev), dev,
                                                   static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_downcast_f32_fp8(const float* src, uint8_t* dst, uint64_t n, sr_fp8_format format, uint64_t seed,
                              uint32_t step, uint32_t tensor_id, uint64_t elem_offset, void* stream) {
    if (format != SR_FP8_E4M3 && format != SR_FP8_E5M2) return SR_ERR_INVALID_ARG;
    if (n == 0) return SR_OK;
    if (src == nullptr || dst == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_downcast_fp8(src, dst, n, format == SR_FP8_E5M2, elem_offset, tensor_id,
                                              static_cast<uint32_t>(seed >> 32), make_keys(seed, step), dev,
                                              static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_downcast_f32_fp4(const float* src, uint8_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                              uint32_t tensor_id, uint64_t elem_offset, void* stream) {
    if (n == 0) return SR_OK;
    if (src == nullptr || dst == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_downcast_fp4(src, dst, n, elem_offset, tensor_id, static_cast<uint32_t>(seed >> 32),
                                              make_keys(seed, step), dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_accumulate_bf16(uint16_t* acc, const void* g, sr_dtype g_dtype, uint64_t n, float scale, uint32_t flags,
                             uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t elem_offset, void* stream) {
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if ((flags & ~static_cast<uint32_t>(SR_FLAG_SR_P)) != 0 || !std::isfinite(scale)) return SR_ERR_INVALID_ARG;
    if (n == 0) return SR_OK;
    if (acc == nullptr || g == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_accumulate(acc, g, g_dtype == SR_DT_F32, n, scale, (flags & SR_FLAG_SR_P) != 0, elem_offset,
                                            tensor_id, static_cast<uint32_t>(seed >> 32), make_keys(seed, step), dev,
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_adamw_step(uint16_t* p, const void* g, sr_dtype g_dtype, uint16_t* m, uint16_t* v, uint64_t n,
                        const sr_adamw_hparams* hp, uint64_t seed, uint32_t step, uint32_t tensor_id,
                        uint64_t elem_offset, void* stream) {
    StepScalars S;
    sr_status st = make_scalars(hp, step, &S);
    if (st != SR_OK) return st;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (n == 0) return SR_OK;
    if (p == nullptr || g == nullptr || m == nullptr || v == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e =
        launch_adamw_flat(p, g, g_dtype == SR_DT_F32, m, v, n, elem_offset, tensor_id, static_cast<uint32_t>(seed >> 32),
                          hp->flags, make_keys(seed, step), S, dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_master_adamw_step(float* p, uint16_t* p_bf16, const void* g, sr_dtype g_dtype, float* m, float* v,
                               uint64_t n, const sr_adamw_hparams* hp, uint32_t step, void* stream) {
    StepScalars S;
    sr_status st = make_scalars(hp, step, &S);
    if (st != SR_OK) return st;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (n == 0) return SR_OK;
    if (p == nullptr || p_bf16 == nullptr || g == nullptr || m == nullptr || v == nullptr) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_master_adamw(p, p_bf16, g, g_dtype == SR_DT_F32, m, v, n, S, dev,
                                              static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

// ---- host-resident state -------------------------------------------------------------------
namespace {
struct HostPipe {
    bool ready = false;
    cudaStream_t side = nullptr;     // second stream of the two-deep pipeline
    cudaEvent_t fork = nullptr, join = nullptr;
};
HostPipe g_pipes[kMaxDevices];
std::mutex g_pipe_mutex;   // the side stream and its two events are shared by all calls on a device

size_t slot_bytes(bool g_f32, uint64_t chunk) {
    // p, m, v (2 bytes each) and g, each region rounded up to 256 bytes
    auto up = [](uint64_t b) { return (b + 255u) & ~static_cast<uint64_t>(255u); };
    return static_cast<size_t>(3 * up(chunk * 2) + up(chunk * (g_f32 ? 4 : 2)));
}
}  // namespace

size_t sr_adamw_step_host_staging_bytes(sr_dtype g_dtype, uint64_t chunk_elems) {
    return 2 * slot_bytes(g_dtype == SR_DT_F32, chunk_elems);
}

sr_status sr_adamw_step_host(uint16_t* p_host, const void* g_host, sr_dtype g_dtype, uint16_t* m_host,
                             uint16_t* v_host, uint64_t n, const sr_adamw_hparams* hp, uint64_t seed, uint32_t step,
                             uint32_t tensor_id, uint64_t elem_offset, void* staging, size_t staging_bytes,
                             uint64_t chunk_elems, void* stream) {
    StepScalars S;
    sr_status st = make_scalars(hp, step, &S);
    if (st != SR_OK) return st;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (n == 0) return SR_OK;
    if (p_host == nullptr || g_host == nullptr || m_host == nullptr || v_host == nullptr) return SR_ERR_INVALID_ARG;
    if (chunk_elems == 0 || (chunk_elems & 7u)) return SR_ERR_INVALID_ARG;
    const bool g_f32 = g_dtype == SR_DT_F32;
    if (staging == nullptr || (reinterpret_cast<uintptr_t>(staging) & 255u) ||
        staging_bytes < sr_adamw_step_host_staging_bytes(g_dtype, chunk_elems))
        return SR_ERR_WORKSPACE;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != SR_OK) return st;
    int dev_id = 0;
    cudaGetDevice(&dev_id);
    std::lock_guard<std::mutex> lock(g_pipe_mutex);   // enqueueing only; nothing below waits for the GPU
    HostPipe& pipe = g_pipes[dev_id];
    cudaError_t e;
    if (!pipe.ready) {
        // all three objects or none: a partial set is destroyed, so a later call starts from scratch
        cudaStream_t side = nullptr;
        cudaEvent_t fork = nullptr, join = nullptr;
        if ((e = cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking)) == cudaSuccess &&
            (e = cudaEventCreateWithFlags(&fork, cudaEventDisableTiming)) == cudaSuccess)
            e = cudaEventCreateWithFlags(&join, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            if (join) cudaEventDestroy(join);
            if (fork) cudaEventDestroy(fork);
            if (side) cudaStreamDestroy(side);
            return cuda_fail(e);
        }
        pipe.side = side;
        pipe.fork = fork;
        pipe.join = join;
        pipe.ready = true;
    }
    cudaStream_t streams[2] = {static_cast<cudaStream_t>(stream), pipe.side};
    // the side stream starts after whatever the caller queued before this call
    if ((e = cudaEventRecord(pipe.fork, streams[0])) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(pipe.side, pipe.fork, 0)) != cudaSuccess) return cuda_fail(e);
    // From here on the side stream is forked off the caller's: every return, failures included, joins it
    // back, so that work queued on the caller's stream afterwards is ordered behind everything enqueued here.
    auto join_side = [&]() -> cudaError_t {
        cudaError_t j = cudaEventRecord(pipe.join, pipe.side);
        if (j == cudaSuccess) j = cudaStreamWaitEvent(streams[0], pipe.join, 0);
        return j;
    };
    auto fail = [&](cudaError_t err) -> sr_status {
        join_side();
        return cuda_fail(err);
    };

    const PhiloxKeys K = make_keys(seed, step);
    const uint32_t seed_hi = static_cast<uint32_t>(seed >> 32);
    const size_t gsz = g_f32 ? 4 : 2;
    const size_t slot = slot_bytes(g_f32, chunk_elems);
    const size_t region = ((chunk_elems * 2 + 255u) / 256u) * 256u;
    uint64_t k = 0;
    for (uint64_t start = 0; start < n; start += chunk_elems, ++k) {
        const uint64_t len = n - start < chunk_elems ? n - start : chunk_elems;
        cudaStream_t s = streams[k & 1u];
        char* base = static_cast<char*>(staging) + (k & 1u) * slot;
        uint16_t* dp = reinterpret_cast<uint16_t*>(base);
        uint16_t* dm = reinterpret_cast<uint16_t*>(base + region);
        uint16_t* dv = reinterpret_cast<uint16_t*>(base + 2 * region);
        void* dg = base + 3 * region;
        const char* gh = static_cast<const char*>(g_host) + start * gsz;
        if ((e = cudaMemcpyAsync(dp, p_host + start, len * 2, cudaMemcpyHostToDevice, s)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(dg, gh, len * gsz, cudaMemcpyHostToDevice, s)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(dm, m_host + start, len * 2, cudaMemcpyHostToDevice, s)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(dv, v_host + start, len * 2, cudaMemcpyHostToDevice, s)) != cudaSuccess) return fail(e);
        e = launch_adamw_flat(dp, dg, g_f32, dm, dv, len, elem_offset + start, tensor_id, seed_hi, hp->flags, K, S, dev, s);
        if (e != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(p_host + start, dp, len * 2, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(m_host + start, dm, len * 2, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(v_host + start, dv, len * 2, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return fail(e);
    }
    // the caller's stream finishes only after the side stream has
    if ((e = join_side()) != cudaSuccess) return cuda_fail(e);
    return SR_OK;
}

sr_status sr_mt_plan_create(sr_mt_plan** out, uint32_t num_tensors, uint16_t* const* p, const void* const* g,
                            uint16_t* const* m, uint16_t* const* v, const uint64_t* numel, sr_dtype g_dtype,
                            void* stream) {
    if (out == nullptr) return SR_ERR_INVALID_ARG;
    *out = nullptr;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (num_tensors != 0 && (p == nullptr || g == nullptr || m == nullptr || v == nullptr || numel == nullptr))
        return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;

    if (num_tensors > 0x7FFFFFFFu) return SR_ERR_INVALID_ARG;
    const size_t gsz = g_dtype == SR_DT_F32 ? 4 : 2;
    std::vector<MtWork> chunks, small;
    std::vector<LargeTensor> large;
    uint64_t total = 0;
    try {
    for (uint32_t i = 0; i < num_tensors; ++i) {
        if (numel[i] != 0 && (p[i] == nullptr || g[i] == nullptr || m[i] == nullptr || v[i] == nullptr))
            return SR_ERR_INVALID_ARG;
        const uint64_t nchunks = (numel[i] + kMtChunkElems - 1) / kMtChunkElems;
        if (chunks.size() + nchunks > 0xFFFFFFFFull) return SR_ERR_INVALID_ARG;
        const uintptr_t bits = reinterpret_cast<uintptr_t>(p[i]) | reinterpret_cast<uintptr_t>(g[i]) |
                               reinterpret_cast<uintptr_t>(m[i]) | reinterpret_cast<uintptr_t>(v[i]);
        const uint32_t tensor_vec = i | ((bits & 15u) == 0 ? 0x80000000u : 0u);
        const bool flat = (bits & 15u) == 0 && numel[i] >= kMtFlatElems;
        if (flat) large.push_back(LargeTensor{p[i], g[i], m[i], v[i], numel[i], i});
        for (uint64_t c = 0; c < nchunks; ++c) {
            const uint64_t start = c * kMtChunkElems;
            const uint64_t left = numel[i] - start;
            const MtWork w{p[i] + start, static_cast<const char*>(g[i]) + start * gsz, m[i] + start, v[i] + start,
                           start, static_cast<uint32_t>(left < kMtChunkElems ? left : kMtChunkElems), tensor_vec};
            chunks.push_back(w);
            if (!flat) small.push_back(w);
        }
        total += numel[i];
    }
    } catch (const std::bad_alloc&) {   // no exception crosses the C ABI
        return SR_ERR_WORKSPACE;
    }

    sr_mt_plan* plan = new (std::nothrow) sr_mt_plan;
    if (plan == nullptr) return SR_ERR_WORKSPACE;
    plan->num_tensors = num_tensors;
    plan->num_chunks = static_cast<uint32_t>(chunks.size());
    plan->total_elements = total;
    plan->g_f32 = g_dtype == SR_DT_F32;
    cudaGetDevice(&plan->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    plan->num_small = static_cast<uint32_t>(small.size());
    try {
        plan->large = std::move(large);
    } catch (const std::bad_alloc&) {
        delete plan;
        return SR_ERR_WORKSPACE;
    }
    if (!chunks.empty()) {
        // one allocation: the full table, then the table of the list kernel's share
        e = cudaMalloc(&plan->d_work, (chunks.size() + small.size()) * sizeof(MtWork));
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(plan->d_work, chunks.data(), chunks.size() * sizeof(MtWork), cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && !small.empty()) {
            plan->d_small = plan->d_work + chunks.size();
            e = cudaMemcpyAsync(plan->d_small, small.data(), small.size() * sizeof(MtWork), cudaMemcpyHostToDevice, s);
        }
        // the host vectors die at return: wait for the copies (plan creation is not a hot call)
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    }
    if (e == cudaSuccess && plan->large.size() >= 2) {
        e = cudaStreamCreateWithFlags(&plan->side, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->join, cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        release_plan(plan);
        return cuda_fail(e);
    }
    *out = plan;
    return SR_OK;
}

sr_status sr_adamw_multi_tensor(const sr_mt_plan* plan, const sr_adamw_hparams* hp, uint64_t seed, uint32_t step,
                                uint32_t tensor_id_base, void* stream) {
    if (plan == nullptr) return SR_ERR_INVALID_ARG;
    StepScalars S;
    sr_status st = make_scalars(hp, step, &S);
    if (st != SR_OK) return st;
    if (plan->num_chunks == 0) return SR_OK;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != SR_OK) return st;
    int current = -1;
    cudaGetDevice(&current);
    if (current != plan->device) return SR_ERR_INVALID_ARG;   // the work table lives on the plan's device
    // large tensors: one flat launch each (index restarts at 0 in every tensor, the tensor id is base + list index:
    // the same noise as in the list kernel); all the others: one launch of the list kernel
    const PhiloxKeys K = make_keys(seed, step);
    const uint32_t seed_hi = static_cast<uint32_t>(seed >> 32);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool two = plan->side != nullptr;
    cudaError_t e = cudaSuccess;
    if (two) {
        e = cudaEventRecord(plan->fork, s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(plan->side, plan->fork, 0);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    size_t turn = 0;
    for (const LargeTensor& t : plan->large) {
        e = launch_adamw_flat(t.p, t.g, plan->g_f32, t.m, t.v, t.numel, 0, tensor_id_base + t.index, seed_hi, hp->flags, K, S,
                              dev, (two && (turn++ & 1u)) ? plan->side : s);
        if (e != cudaSuccess) break;
    }
    if (two) {   // joined on every path: the side stream never stays forked from the caller's
        cudaError_t j = cudaEventRecord(plan->join, plan->side);
        if (j == cudaSuccess) j = cudaStreamWaitEvent(s, plan->join, 0);
        if (e == cudaSuccess) e = j;
    }
    // the list kernel after the join: its blocks would share SMs with a flat launch's (one flat launch beside the list
    // kernel on the GPT-2 350M list: 0.805 -> 0.822 ms), whereas two flat launches cannot share an SM
    if (e == cudaSuccess && plan->num_small != 0)
        e = launch_adamw_mt(plan->d_small, plan->num_small, plan->g_f32, tensor_id_base, seed_hi, hp->flags, K, S, dev, s);
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_mt_plan_destroy(sr_mt_plan* plan) {
    if (plan == nullptr) return SR_OK;
    const cudaError_t e = release_plan(plan);
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

uint64_t sr_mt_plan_total_elements(const sr_mt_plan* plan) { return plan ? plan->total_elements : 0; }

size_t grad_sqnorm_workspace_bytes(uint64_t n) { return static_cast<size_t>(sqnorm_scratch_doubles(n) * sizeof(double)); }

sr_status grad_sqnorm(const void* g, sr_dtype g_dtype, uint64_t n, double* out_dev, void* workspace,
                      size_t workspace_bytes, void* stream) {
    if (out_dev == nullptr) return SR_ERR_INVALID_ARG;
    if (g_dtype != SR_DT_BF16 && g_dtype != SR_DT_F32) return SR_ERR_INVALID_ARG;
    if (n != 0 && g == nullptr) return SR_ERR_INVALID_ARG;
    const size_t need = grad_sqnorm_workspace_bytes(n);
    if (need != 0 && (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 7u)))
        return SR_ERR_WORKSPACE;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_sqnorm(g, g_dtype == SR_DT_F32, n, out_dev, static_cast<double*>(workspace), dev,
                                        static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

size_t grad_sqnorm_multi_tensor_workspace_bytes(const sr_mt_plan* plan) {
    return plan ? static_cast<size_t>(sqnorm_mt_scratch_doubles(plan->num_chunks) * sizeof(double)) : 0;
}

sr_status grad_sqnorm_multi_tensor(const sr_mt_plan* plan, double* out_dev, void* workspace, size_t workspace_bytes,
                                   void* stream) {
    if (plan == nullptr || out_dev == nullptr) return SR_ERR_INVALID_ARG;
    const size_t need = grad_sqnorm_multi_tensor_workspace_bytes(plan);
    if (need != 0 && (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 7u)))
        return SR_ERR_WORKSPACE;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    int current = -1;
    cudaGetDevice(&current);
    if (current != plan->device) return SR_ERR_INVALID_ARG;
    const cudaError_t e = launch_sqnorm_mt(plan->d_work, plan->num_chunks, plan->g_f32, out_dev,
                                           static_cast<double*>(workspace), dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

sr_status sr_clip_scale(const double* sqnorm_dev, float accum_scale, float max_norm, float* gscale_out_dev,
                        void* stream) {
    if (sqnorm_dev == nullptr || gscale_out_dev == nullptr) return SR_ERR_INVALID_ARG;
    if (!finite_f(accum_scale) || !finite_f(max_norm) || max_norm < 0.0f) return SR_ERR_INVALID_ARG;
    DeviceInfo dev;
    sr_status st = current_device(&dev);
    if (st != SR_OK) return st;
    const cudaError_t e = launch_clip_scale(sqnorm_dev, accum_scale, max_norm, gscale_out_dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SR_OK : cuda_fail(e);
}

const char* sr_status_string(sr_status s) {
    switch (s) {
        case SR_OK: return "ok";
        case SR_ERR_INVALID_ARG: return "invalid argument";
        case SR_ERR_UNSUPPORTED_DEVICE: return "unsupported device (compute capability 10.x required)";
        case SR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SR_ERR_CUDA: return "CUDA runtime error (see sr_last_cuda_error)";
    }
    return "unknown status";
}

int sr_last_cuda_error(void) { return tl_last_cuda_error; }

uint32_t sr_abi_version(void) { return SR_ABI_VERSION; }

}  // extern "C"
