// mqa_decode_static: the decode step for callers that cannot allocate device memory.
//
// Some callers have no way to obtain a workspace: code that runs where cudaMalloc
// is forbidden or unavailable (a plugin inside a host application that owns all
// device memory and hands none out, a latency-critical serving loop that must not
// touch the allocator, an environment where allocation calls are stubbed out).
// For them the scratch that mqa_decode normally receives from the caller lives
// here, in a fixed array in the library's own device image.  Every GPU that loads
// the library pays for this array until the process exits, so it is kept modest
// and shapes that would need more are rejected.
//
// All calls on a device share the one array, and the array keeps whatever the last
// call left in it.  The parts that must start clean (the header with the device status
// word, the per-sequence records and arrival counters) are cleared by each call on its
// stream before launching.  Two calls
// whose kernels overlap on the GPU (different streams, no ordering) would race on
// the array: callers must order them.
#include "../../include/mqa_decode.h"
#include "mqa_common.cuh"

#include <mutex>

namespace {

constexpr size_t kStaticBytes = (size_t)MQA_STATIC_WORKSPACE_BYTES;

// The scratch itself.  In host code this name is only a handle for the runtime's
// symbol lookup, not a device address; kernels must be given the address that
// cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_device_ptr[kMaxDevices] = {};

// Device address of the array on the current device, looked up once per device.
int static_workspace(unsigned char** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return MQA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_device_ptr[dev]) {
        unsigned char* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_workspace) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_device_ptr[dev] = ptr;
    }
    *out = g_device_ptr[dev];
    return MQA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int mqa_decode_static(const void* q, const void* k_cache, const void* v_cache,
                                 const int32_t* lengths, float* out,
                                 int B, int H, int D, int Lmax, float scale, void* stream)
{
    if (!q || !k_cache || !v_cache || !lengths || !out) return MQA_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0 || !(scale == scale)) return MQA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return MQA_ERR_MISALIGNED;

    mqa_plan_t plan;
    int rc = mqa_decode_plan(B, H, D, Lmax, MQA_PATH_AUTO, &plan);   // host arithmetic only
    if (rc != MQA_OK) return rc;

    // Fit the plan into the fixed array: header + per-sequence records + two slots per block.
    const size_t fixed = mqa::slots_offset(B);
    const size_t slot_bytes = mqa::slot_floats(H, D) * sizeof(float);
    if (fixed + 2 * slot_bytes > kStaticBytes) return MQA_ERR_WORKSPACE_TOO_SMALL;   // B (or H*D) beyond the maximum
    const size_t fit = (kStaticBytes - fixed) / (2 * slot_bytes);
    if ((size_t)plan.num_ctas > fit) plan.num_ctas = (int)fit;

    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    if (major != 10) return MQA_ERR_ARCH;

    unsigned char* ws = nullptr;
    rc = static_workspace(&ws);
    if (rc != MQA_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents; the header, the per-sequence records and the arrival
    // counters (everything in front of the partial-result slots) have to start at zero.
    if (cudaMemsetAsync(ws, 0, fixed, st) != cudaSuccess) return MQA_ERR_CUDA;

    mqa::Params p;
    p.q = static_cast<const uint16_t*>(q);
    p.k = static_cast<const uint16_t*>(k_cache);
    p.v = static_cast<const uint16_t*>(v_cache);
    p.lengths = mqa::LenView{lengths, 1};
    p.out = out;
    p.n_dst = 0; p.b_offset = 0;
    for (int r = 0; r < mqa::kMaxDst; ++r) p.out_dst[r] = nullptr;
    p.B = B; p.H = H; p.D = D; p.Lmax = Lmax;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.tile_shift = (plan.tile_rows == 128) ? 7 : 6;
    p.num_ctas = plan.num_ctas;
    p.adaptive = (plan.path == MQA_PATH_TC) ? plan.adaptive : 0;
    p.cluster = 1;
    p.lo_max_len = 0x7fffffff;
    p.workspace = ws;
    cudaError_t e = (plan.path == MQA_PATH_TC) ? mqa::launch_tc(p, st) : mqa::launch_fma(p, st);
    if (e != cudaSuccess) return MQA_ERR_CUDA;
    if (plan.path != MQA_PATH_TC && mqa::launch_combine(p, st) != cudaSuccess) return MQA_ERR_CUDA;
    return MQA_OK;
}
