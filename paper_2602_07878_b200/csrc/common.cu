// Host-side helpers shared by the entry points: error slots, device info, shape checks.
#include <atomic>
#include <mutex>

#include "internal.h"
#include "ptx.cuh"

namespace pk {

static thread_local int tl_cuda_error = 0;
static std::atomic<int64_t> g_launches{0};

void set_cuda_error(int code) { tl_cuda_error = code; }

int check_cuda(cudaError_t e) {
    if (e == cudaSuccess) return PA_OK;
    tl_cuda_error = static_cast<int>(e);
    return PA_ERR_CUDA;
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int get_device_info(DeviceInfo* info) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    static bool have[64] = {false};
    int dev = 0;
    int rc = check_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    std::lock_guard<std::mutex> lk(mu);
    if (dev < 0 || dev >= 64) return PA_ERR_ARG;
    if (!have[dev]) {
        DeviceInfo d;
        d.device = dev;
        rc = check_cuda(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
        if (rc) return rc;
        rc = check_cuda(
            cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        if (rc) return rc;
        cache[dev] = d;
        have[dev] = true;
    }
    *info = cache[dev];
    return PA_OK;
}

int validate_shape(const pa_shape* s) {
    if (s->dtype != PA_BF16) return PA_ERR_SHAPE;
    if (s->head_dim != 64 && s->head_dim != 128 && s->head_dim != 256) return PA_ERR_SHAPE;
    if (s->block_size != BS) return PA_ERR_SHAPE;
    if (s->num_kv_heads <= 0 || s->num_q_heads <= 0) return PA_ERR_SHAPE;
    if (s->num_q_heads % s->num_kv_heads) return PA_ERR_SHAPE;
    if (s->num_q_heads / s->num_kv_heads > 16) return PA_ERR_SHAPE;
    if (s->num_blocks <= 0) return PA_ERR_SHAPE;
    const int64_t st[3] = {s->stride_block, s->stride_head, s->stride_tok};
    for (int i = 0; i < 3; ++i)
        if (st[i] <= 0 || st[i] % 8 || st[i] >= (int64_t(1) << 38)) return PA_ERR_SHAPE;
    if (s->stride_tok < s->head_dim) return PA_ERR_SHAPE;
    return PA_OK;
}

}  // namespace pk

namespace pk {
// One warp waits, with the same bounded wait the attention kernels use, on a barrier that
// nobody will ever complete.  When the limit passes it reports PA_STATUS_TIMEOUT and returns.
__global__ void wait_expiry_kernel(unsigned long long limit_ns, int* status) {
    __shared__ __align__(8) unsigned long long barrier_word;
    const uint32_t bar = smem_u32(&barrier_word);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
    }
    __syncwarp();
    if (!mbar_wait_bounded(bar, 0, limit_ns) && threadIdx.x == 0)
        atomicOr(status, PA_STATUS_TIMEOUT);
}
}  // namespace pk

extern "C" int pa_selftest_wait_expiry(int32_t limit_us, int32_t* dev_status, void* cuda_stream) {
    if (!dev_status) return PA_ERR_NULL;
    if (limit_us <= 0 || limit_us > 100000) return PA_ERR_ARG;  // at most 0.1 s
    pk::wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        (unsigned long long)limit_us * 1000ull, dev_status);
    pk::count_launch();
    return pk::check_cuda(cudaGetLastError());
}

extern "C" const char* pa_status_string(int code) {
    switch (code) {
        case PA_OK: return "ok";
        case PA_ERR_NULL: return "a required pointer is NULL";
        case PA_ERR_SHAPE: return "unsupported shape, dtype or strides";
        case PA_ERR_ALIGN: return "buffer not sufficiently aligned";
        case PA_ERR_WORKSPACE: return "workspace or staging buffer too small";
        case PA_ERR_HOSTBUF: return "host buffer too small or not pinned";
        case PA_ERR_BLOCK_ID: return "block id out of range or duplicated";
        case PA_ERR_CUDA: return "CUDA call failed (see pa_last_cuda_error)";
        case PA_ERR_ARG: return "invalid argument";
        case PA_ERR_STATIC_LIMIT:
            return "request needs more scratch than the built-in static workspace holds";
        default: return "unknown status";
    }
}

extern "C" int pa_last_cuda_error(void) { return pk::tl_cuda_error; }

extern "C" int64_t pa_launch_count(void) { return pk::g_launches.load(); }
