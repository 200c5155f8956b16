// fp32-FMA multiquery decode kernel: the path for small H*D and the fallback for
// every supported shape.  One persistent block walks its run of K/V tiles
// (64 cache rows each); each tile is staged into shared memory once and used by
// all H query heads, which is the multiquery saving of the paper's Section 3.3.
// Per tile: logits (fp32 FMA) -> mask -> base-2 online softmax -> weighted V sum.
#include "mqa_common.cuh"

namespace mqa {

constexpr int kFmaThreads = 256;
constexpr int kFmaTileShift = 6;
constexpr int kFmaTile = 1 << kFmaTileShift;
constexpr int kSStride = kFmaTile + 1;     // fp32 logits/probabilities row stride (bank spread)

template <int D>
struct FmaSmem {
    static constexpr int kKStride = D + 8;                 // bf16 elements; 16 B pad spreads banks
    static constexpr size_t kK = (size_t)kFmaTile * kKStride * 2;
    static constexpr size_t kV = (size_t)kFmaTile * D * 2;
    __host__ __device__ static constexpr size_t q_bytes(int H) { return (size_t)H * D * 2; }
    __host__ __device__ static constexpr size_t s_bytes(int H) { return (size_t)H * kSStride * 4; }
    static size_t total(int H) {
        return kK + kV + q_bytes(H) + s_bytes(H) + 3 * kMaxHeads * sizeof(float) + sizeof(SchedShared) + 64;
    }
};

template <int D>
__global__ void __launch_bounds__(kFmaThreads)
mqa_fma_kernel(const Params p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using SM = FmaSmem<D>;
    constexpr int KS = SM::kKStride;
    uint16_t* sK = reinterpret_cast<uint16_t*>(smem_raw);
    uint16_t* sV = reinterpret_cast<uint16_t*>(smem_raw + SM::kK);
    uint16_t* sQ = reinterpret_cast<uint16_t*>(smem_raw + SM::kK + SM::kV);
    float* sS = reinterpret_cast<float*>(smem_raw + SM::kK + SM::kV + SM::q_bytes(p.H));
    float* sM = sS + (size_t)p.H * kSStride;
    float* sL = sM + kMaxHeads;
    float* sAlpha = sL + kMaxHeads;
    // 8-byte aligned (the record holds 64-bit tile indices; the row stride above is odd): total() reserves the slack
    SchedShared& sched = *reinterpret_cast<SchedShared*>((reinterpret_cast<uintptr_t>(sAlpha + kMaxHeads) + 7) & ~uintptr_t(7));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = p.H, cta = blockIdx.x, G = p.num_ctas;

    const int T = schedule_prologue<kFmaThreads>(p.lengths, p.B, p.Lmax, kFmaTileShift, G, cta, sched);
    if (cta == 0 && tid == 0) {
        ws_header(p.workspace)[kHdrTotalTiles] = T;
        ws_header(p.workspace)[kHdrNumCtas] = G;
    }
    if (T == 0) return;
    SegmentWalker w;
    w.init(p.lengths, p.B, p.Lmax, kFmaTileShift, T, G, cta, sched.b0, sched.p0);

    // thread roles
    const int l_pos = tid & (kFmaTile - 1);     // logits: cache row within the tile
    const int hg = tid >> kFmaTileShift;        // logits: head group 0..3 (heads hg, hg+4, ...)
    constexpr int TPD = D / 8;                  // PV: threads across D (8 columns each)
    constexpr int HG2 = kFmaThreads / TPD;      // PV: head groups
    constexpr int HPT2 = (kMaxHeads + HG2 - 1) / HG2;
    const int dq = tid % TPD, hg2 = tid / TPD;

    for (; !w.done(); w.next()) {
        const int b = w.b, len = w.len;
        const int t0 = w.seg_t0(), t1 = w.seg_t1();
        const bool whole = w.seg_is_whole();
        if (w.seg_owns_first_tile() && tid == 0) {
            SeqInfo si;
            si.first_slot = whole ? -1 : w.seg_slot(cta);
            si.last_cta = cta_of_tile(w.P + w.nt - 1, T, G);
            ws_seqinfo(p.workspace)[b] = si;
        }
        __syncthreads();   // previous segment finished with sQ/sM/sL
        {   // stage q[b] and reset the running statistics
            const uint4* src = reinterpret_cast<const uint4*>(p.q + (size_t)b * H * D);
            uint4* dst = reinterpret_cast<uint4*>(sQ);
            for (int i = tid; i < H * D / 8; i += kFmaThreads) dst[i] = __ldg(src + i);
            if (tid < H) { sM[tid] = -INFINITY; sL[tid] = 0.f; }
        }
        float acc[HPT2][8];
#pragma unroll
        for (int i = 0; i < HPT2; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

        for (int t = t0; t < t1; ++t) {
            const int row0 = t << kFmaTileShift;
            const int nvalid = min(kFmaTile, len - row0);
            __syncthreads();   // previous tile's consumers are done with sK/sV/sS
            {
                const uint4* gk = reinterpret_cast<const uint4*>(p.k + ((size_t)b * p.Lmax + row0) * D);
                const uint4* gv = reinterpret_cast<const uint4*>(p.v + ((size_t)b * p.Lmax + row0) * D);
                uint4* dk = reinterpret_cast<uint4*>(sK);
                uint4* dv = reinterpret_cast<uint4*>(sV);
                for (int i = tid; i < nvalid * TPD; i += kFmaThreads) {
                    const int r = i / TPD, c = i % TPD;
                    dk[r * (KS / 8) + c] = __ldcs(gk + i);
                    dv[i] = __ldcs(gv + i);
                }
            }
            __syncthreads();
            // ---- logits: s[h,l] = scale_log2 * q[h,:].k[l,:], masked beyond the length ----
            {
                constexpr int HPT = kMaxHeads / 4;
                float s[HPT];
#pragma unroll
                for (int i = 0; i < HPT; ++i) s[i] = 0.f;
                if (l_pos < nvalid) {
                    const uint4* krow = reinterpret_cast<const uint4*>(sK + (size_t)l_pos * KS);
#pragma unroll 2
                    for (int c = 0; c < TPD; ++c) {
                        const uint4 kk = krow[c];
                        const float k0 = bf16_lo(kk.x), k1 = bf16_hi(kk.x), k2 = bf16_lo(kk.y), k3 = bf16_hi(kk.y);
                        const float k4 = bf16_lo(kk.z), k5 = bf16_hi(kk.z), k6 = bf16_lo(kk.w), k7 = bf16_hi(kk.w);
#pragma unroll
                        for (int i = 0; i < HPT; ++i) {
                            const int h = hg + 4 * i;
                            if (h < H) {
                                const uint4 qq = reinterpret_cast<const uint4*>(sQ + (size_t)h * D)[c];
                                float a = s[i];
                                a = fmaf(bf16_lo(qq.x), k0, a); a = fmaf(bf16_hi(qq.x), k1, a);
                                a = fmaf(bf16_lo(qq.y), k2, a); a = fmaf(bf16_hi(qq.y), k3, a);
                                a = fmaf(bf16_lo(qq.z), k4, a); a = fmaf(bf16_hi(qq.z), k5, a);
                                a = fmaf(bf16_lo(qq.w), k6, a); a = fmaf(bf16_hi(qq.w), k7, a);
                                s[i] = a;
                            }
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < HPT; ++i) {
                    const int h = hg + 4 * i;
                    if (h < H) sS[h * kSStride + l_pos] = (l_pos < nvalid) ? s[i] * p.scale_log2 : -INFINITY;
                }
            }
            __syncthreads();
            // ---- online softmax, one warp per head ----
            for (int h = warp; h < H; h += kFmaThreads / 32) {
                float* row = sS + h * kSStride;
                const float s0 = row[lane], s1 = row[lane + 32];
                float mx = fmaxf(s0, s1);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_old = sM[h];
                const float m_new = fmaxf(m_old, mx);          // finite: every tile has a valid row
                const float p0 = exp2f(s0 - m_new), p1 = exp2f(s1 - m_new);
                row[lane] = p0; row[lane + 32] = p1;
                float sum = p0 + p1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                if (lane == 0) {
                    const float alpha = exp2f(m_old - m_new);   // 0 on the first tile (m_old = -inf)
                    sAlpha[h] = alpha;
                    sM[h] = m_new;
                    sL[h] = sL[h] * alpha + sum;
                }
            }
            __syncthreads();
            // ---- weighted values: acc[h, d] = alpha*acc + sum_l p[h,l] v[l,d] ----
#pragma unroll
            for (int i = 0; i < HPT2; ++i) {
                const int h = hg2 + HG2 * i;
                if (h < H) {
                    const float a = sAlpha[h];
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] *= a;
                }
            }
            for (int l = 0; l < nvalid; ++l) {
                const uint4 vv = reinterpret_cast<const uint4*>(sV + (size_t)l * D)[dq];
                const float v0 = bf16_lo(vv.x), v1 = bf16_hi(vv.x), v2 = bf16_lo(vv.y), v3 = bf16_hi(vv.y);
                const float v4 = bf16_lo(vv.z), v5 = bf16_hi(vv.z), v6 = bf16_lo(vv.w), v7 = bf16_hi(vv.w);
#pragma unroll
                for (int i = 0; i < HPT2; ++i) {
                    const int h = hg2 + HG2 * i;
                    if (h < H) {
                        const float pr = sS[h * kSStride + l];
                        acc[i][0] = fmaf(pr, v0, acc[i][0]); acc[i][1] = fmaf(pr, v1, acc[i][1]);
                        acc[i][2] = fmaf(pr, v2, acc[i][2]); acc[i][3] = fmaf(pr, v3, acc[i][3]);
                        acc[i][4] = fmaf(pr, v4, acc[i][4]); acc[i][5] = fmaf(pr, v5, acc[i][5]);
                        acc[i][6] = fmaf(pr, v6, acc[i][6]); acc[i][7] = fmaf(pr, v7, acc[i][7]);
                    }
                }
            }
        }
        // ---- segment epilogue ----
        float* slot = whole ? nullptr : ws_slot(p.workspace, p.B, H, D, w.seg_slot(cta));
        const int Hp4 = round_up(H, 4);
        if (!whole && tid < H) { slot[tid] = sM[tid]; slot[Hp4 + tid] = sL[tid]; }
#pragma unroll
        for (int i = 0; i < HPT2; ++i) {
            const int h = hg2 + HG2 * i;
            if (h < H) {
                float4 a, c;
                if (whole) {
                    const float inv = 1.f / sL[h];
                    a = make_float4(acc[i][0] * inv, acc[i][1] * inv, acc[i][2] * inv, acc[i][3] * inv);
                    c = make_float4(acc[i][4] * inv, acc[i][5] * inv, acc[i][6] * inv, acc[i][7] * inv);
                    float4* dst = reinterpret_cast<float4*>(p.out + ((size_t)b * H + h) * D + dq * 8);
                    dst[0] = a; dst[1] = c;
                } else {
                    a = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                    c = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
                    float4* dst = reinterpret_cast<float4*>(slot + 2 * Hp4 + (size_t)h * D + dq * 8);
                    dst[0] = a; dst[1] = c;
                }
            }
        }
    }
}

template <int D>
static cudaError_t launch_fma_d(const Params& p, cudaStream_t stream)
{
    const size_t smem = FmaSmem<D>::total(p.H);
    cudaError_t e = cudaFuncSetAttribute(mqa_fma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    mqa_fma_kernel<D><<<p.num_ctas, kFmaThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_fma(const Params& p, cudaStream_t stream)
{
    switch (p.D) {
        case 64: return launch_fma_d<64>(p, stream);
        case 128: return launch_fma_d<128>(p, stream);
        case 256: return launch_fma_d<256>(p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace mqa
