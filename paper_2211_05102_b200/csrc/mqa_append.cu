// Appends the decode step's new key/value row of every sequence to its cache and bumps the length,
// ahead of the attention over the lengthened cache (the generate loop of the paper's Section 2.2:
// each step produces one token per sequence whose K/V joins the cache that the next attention reads;
// Section 3.3: "one token per example of Q, K and V, whereas the KV cache has many").
#include "mqa_common.cuh"

namespace mqa {

// One block per sequence; thread t copies 16 bytes of the K row and 16 bytes of the V row.
__global__ void mqa_append_kernel(const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                                  uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
                                  int32_t* __restrict__ lengths, int D, int Lmax, unsigned char* workspace)
{
    const int b = blockIdx.x;
    const int len = lengths[b];
    if (len < 0 || len >= Lmax) {
        // no room (or a corrupt length): nothing is written, the length stays, the host can see why
        if (threadIdx.x == 0) atomicExch(ws_header(workspace) + kHdrStatus, 8 /* MQA_ERR_CACHE_FULL */);
        return;
    }
    const size_t row = ((size_t)b * Lmax + len) * D;
    for (int i = threadIdx.x; i < D / 8; i += blockDim.x) {
        reinterpret_cast<uint4*>(k_cache + row)[i] = __ldg(reinterpret_cast<const uint4*>(k_new + (size_t)b * D) + i);
        reinterpret_cast<uint4*>(v_cache + row)[i] = __ldg(reinterpret_cast<const uint4*>(v_new + (size_t)b * D) + i);
    }
    __syncthreads();
    if (threadIdx.x == 0) lengths[b] = len + 1;
}

cudaError_t launch_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int32_t* lengths,
                          int B, int D, int Lmax, unsigned char* workspace, cudaStream_t stream)
{
    mqa_append_kernel<<<B, 32, 0, stream>>>(static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),
                                            static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache),
                                            lengths, D, Lmax, workspace);
    return cudaGetLastError();
}

}  // namespace mqa
