// Log-sum-exp combine: merges the partial results of every sequence whose tiles
// were cut across thread blocks, and writes zeros for empty sequences.
//   M = max_s m_s;  out = sum_s 2^(m_s-M) acc_s / sum_s 2^(m_s-M) l_s
// (m_s, l_s are in the base-2 logit domain the split kernels use.)
#include "mqa_common.cuh"

namespace mqa {

constexpr int kCombineThreads = 256;
constexpr int kCombineHeadsPerBlock = kCombineThreads / 32;

__global__ void __launch_bounds__(kCombineThreads)
mqa_combine_kernel(const Params p)
{
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = blockIdx.y * kCombineHeadsPerBlock + warp;
    const int H = p.H, D = p.D;
    if (h >= H) return;
    float* orow = p.out + ((size_t)b * H + h) * D;
    const int len = clamp_len(p.lengths[b], p.Lmax);
    if (len == 0) {
        for (int d = lane * 4; d < D; d += 128) *reinterpret_cast<float4*>(orow + d) = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const SeqInfo si = ws_seqinfo(p.workspace)[b];
    if (si.first_slot < 0) return;                 // a single block wrote the output directly
    const int T = ws_header(p.workspace)[kHdrTotalTiles];
    const int G = p.num_ctas;
    const int Hp4 = round_up(H, 4);
    const int i_first = si.first_slot >> 1;

    // pass 1: the maximum over the sequence's partial results
    float M = ws_slot(p.workspace, p.B, H, D, si.first_slot)[h];
    for (int i = i_first + 1; i <= si.last_cta; ++i) {
        if (span_begin(i, T, G) == span_begin(i + 1, T, G)) continue;   // block without tiles
        M = fmaxf(M, ws_slot(p.workspace, p.B, H, D, 2 * i)[h]);
    }
    // pass 2: weighted sums
    float4 acc[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
    float lsum = 0.f;
    for (int i = i_first; i <= si.last_cta; ++i) {
        if (i > i_first && span_begin(i, T, G) == span_begin(i + 1, T, G)) continue;
        const float* slot = ws_slot(p.workspace, p.B, H, D, i == i_first ? si.first_slot : 2 * i);
        const float wgt = exp2f(slot[h] - M);
        lsum = fmaf(wgt, slot[Hp4 + h], lsum);
        const float* a = slot + 2 * Hp4 + (size_t)h * D;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int d = lane * 4 + j * 128;
            if (d < D) {
                const float4 x = *reinterpret_cast<const float4*>(a + d);
                acc[j].x = fmaf(wgt, x.x, acc[j].x); acc[j].y = fmaf(wgt, x.y, acc[j].y);
                acc[j].z = fmaf(wgt, x.z, acc[j].z); acc[j].w = fmaf(wgt, x.w, acc[j].w);
            }
        }
    }
    const float inv = 1.f / lsum;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int d = lane * 4 + j * 128;
        if (d < D)
            *reinterpret_cast<float4*>(orow + d) = make_float4(acc[j].x * inv, acc[j].y * inv, acc[j].z * inv, acc[j].w * inv);
    }
}

cudaError_t launch_combine(const Params& p, cudaStream_t stream)
{
    dim3 grid(p.B, (p.H + kCombineHeadsPerBlock - 1) / kCombineHeadsPerBlock);
    mqa_combine_kernel<<<grid, kCombineThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace mqa
