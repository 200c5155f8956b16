// Shared device/host declarations of the multiquery decode-attention kernels:
// workspace layout, the flattened tile schedule, and small helpers.
//
// Schedule.  Sequence b owns nt_b = ceil(len_b / tile_rows) tiles of its K/V
// cache; the tiles of all sequences are numbered consecutively (sequence-major)
// from 0 to T-1.  Persistent thread block i of G takes the contiguous run
// [floor(i*T/G), floor((i+1)*T/G)).  A run crosses sequence boundaries; the
// piece of a sequence inside one run is a "segment".  A segment that covers its
// whole sequence writes the normalised output directly; any other segment
// writes a partial result (running max m, running sum l, unnormalised
// accumulator) into one of the block's two slots, and the combine kernel merges
// the partial results of each cut sequence.  Each block recomputes the prefix
// sums of the tile counts itself, so the host never reads `lengths`.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mqa {

constexpr int kHeaderBytes = 256;
constexpr int kMaxCtas = 592;
constexpr int kMaxHeads = 64;
constexpr int kMaxDst = 16;               // destinations of a scattered output (ranks of one NVLink domain)

// Workspace header words (int32).
enum { kHdrStatus = 0, kHdrTotalTiles = 2, kHdrNumCtas = 3, kHdrPairMode = 4 };

// Per-sequence record written by the block that owns the sequence's first tile.
struct SeqInfo {
    int first_slot;   // -1: the output was written directly; else slot index of the first partial
    int last_cta;     // block that owns the sequence's last tile
};

__host__ __device__ inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// A partial-result slot: m[Hp4], l[Hp4], acc[H*D] (fp32), Hp4 = H rounded up to 4.
__host__ __device__ inline size_t slot_floats(int H, int D) {
    return (size_t)2 * round_up(H, 4) + (size_t)H * D;
}
__host__ __device__ inline size_t seqinfo_offset() { return kHeaderBytes; }
// One arrival counter per sequence (tensor-core path: the blocks holding parts of a cut sequence merge it
// together once all parts have arrived).  Zero between calls: the last block to leave the merge resets it.
__host__ __device__ inline size_t arrivals_offset(int B) {
    return kHeaderBytes + ((size_t)B * sizeof(SeqInfo) + 255) / 256 * 256;
}
__host__ __device__ inline size_t slots_offset(int B) {
    return arrivals_offset(B) + ((size_t)B * sizeof(int) + 255) / 256 * 256;
}
__host__ __device__ inline size_t workspace_bytes(int B, int H, int D) {
    return slots_offset(B) + (size_t)2 * kMaxCtas * slot_floats(H, D) * sizeof(float);
}

// Lengths as the kernels see them: entry b of a batch of B*kv_groups "sequences" is lengths[b / kv_groups]
// (every key/value head of a sequence has that sequence's length); kv_groups = 1 for multiquery attention.
struct LenView {
    const int32_t* ptr;
    int groups;
    __host__ __device__ __forceinline__ int operator[](int b) const { return groups == 1 ? ptr[b] : ptr[b / groups]; }
};

struct Params {
    const uint16_t* q;        // bf16 bits [B,H,D]
    const uint16_t* k;        // [B,Lmax,D]
    const uint16_t* v;        // [B,Lmax,D]
    LenView lengths;          // [B / kv_groups] int32, viewed per (sequence, key/value head)
    float* out;               // [B,H,D] (unused when the output is scattered)
    // Scattered output (batch-sharded attention feeding a heads-sharded projection): head h of local sequence b
    // goes to row (b_offset + b) of destination h / (H / n_dst), a [B_total, H / n_dst, D] buffer that may live
    // in a peer GPU's memory.  n_dst = 0: plain output.
    float* out_dst[kMaxDst];
    int n_dst, b_offset;
    int B, H, D, Lmax;
    float scale_log2;         // scale * log2(e): logits are kept in the base-2 domain
    int tile_shift;           // log2(tile_rows)
    int num_ctas;             // G (an upper bound when `adaptive` is set)
    int adaptive;             // tensor-core path: the kernel may run a uniform batch on fewer blocks (uniform_ctas)
    int cluster;              // thread blocks per cluster of this launch (1, or 2: pairs may merge through shared memory)
    int lo_max_len;           // tensor-core path: sequences up to this length use hi+lo bf16 probabilities
    unsigned char* workspace;
};

// Address of output row (b, h): D contiguous floats.
__device__ __forceinline__ float* out_row(const Params& p, int b, int h) {
    if (p.n_dst == 0) return p.out + ((size_t)b * p.H + h) * p.D;
    const int hpd = p.H / p.n_dst, r = h / hpd;
    return p.out_dst[r] + ((size_t)(p.b_offset + b) * hpd + (h - r * hpd)) * p.D;
}

__host__ __device__ __forceinline__ int clamp_len(int len, int Lmax) { return len < 0 ? 0 : (len > Lmax ? Lmax : len); }

__device__ __forceinline__ int* ws_header(unsigned char* ws) { return reinterpret_cast<int*>(ws); }
__device__ __forceinline__ SeqInfo* ws_seqinfo(unsigned char* ws) {
    return reinterpret_cast<SeqInfo*>(ws + seqinfo_offset());
}
__device__ __forceinline__ int* ws_arrivals(unsigned char* ws, int B) {
    return reinterpret_cast<int*>(ws + arrivals_offset(B));
}
__device__ __forceinline__ float* ws_slot(unsigned char* ws, int B, int H, int D, int slot) {
    return reinterpret_cast<float*>(ws + slots_offset(B)) + (size_t)slot * slot_floats(H, D);
}

// First tile of block i's run (0 <= i <= G).  The products are at most T*G: 32-bit arithmetic whenever that
// fits (a 64-bit division is some hundred instructions, and these sit in every launch's prologue).
__host__ __device__ inline long long span_begin(int i, int T, int G) {
    if ((unsigned long long)(unsigned)T * (unsigned)G <= 0xffffffffull) return (long long)((unsigned)i * (unsigned)T / (unsigned)G);
    return (long long)i * T / G;
}
// The block whose run contains tile g (0 <= g < T).
__host__ __device__ inline int cta_of_tile(long long g, int T, int G) {
    if ((unsigned long long)(unsigned)T * (unsigned)G + (unsigned)T <= 0xffffffffull)
        return (int)((((unsigned)g + 1u) * (unsigned)G + (unsigned)T - 1u) / (unsigned)T) - 1;
    return (int)(((g + 1) * G + T - 1) / T) - 1;
}

// Block count for a batch in which every one of the B sequences owns the same number of tiles `nt`.
// With G blocks sharing T = B*nt tiles evenly, almost every block boundary cuts a sequence, and each cut costs
// two partial epilogues and a merge (about 8 us per block in total, measured).  A block count g whose cuts all
// fall on sequence boundaries (g divides B: whole sequences per block) or cut every sequence into the same
// number of equal parts (B divides g and g/B divides nt) avoids most of that; it is chosen when the K/V stream
// is not slowed by more than the saving.  Stream model: one SM sustains a tile per kPerSmTileNs, and about
// kSmsToSaturate of them saturate HBM, so fewer blocks than that stretch the stream proportionally.
__host__ __device__ inline int uniform_ctas(int B, int nt, int G)
{
    constexpr float kPerSmTileNs = 2330.f, kSmsToSaturate = 123.f, kCutSavingNs = 7000.f;
    const long long T = (long long)B * nt;
    if (nt <= 1 || T <= G) return G;                  // one tile per sequence: every cut is on a boundary already
    auto stream_ns = [&](int g) { return (float)T * kPerSmTileNs / (g < kSmsToSaturate ? (float)g : kSmsToSaturate); };
    int cand = 0;
    if (B >= G) {
        // whole sequences per block: the largest divisor of B that is <= G, if it is near G
        const int k0 = (B + G - 1) / G;
        for (int k = k0; k < k0 + 4 && cand == 0; ++k)
            if (B % k == 0) cand = B / k;
    } else {
        // every sequence cut into s equal parts
        const int s0 = G / B;
        for (int s = s0; s >= 1 && s > s0 - 4 && cand == 0; --s)
            if (nt % s == 0) cand = B * s;
    }
    if (cand <= 0 || cand >= G) return G;
    return (stream_ns(cand) - stream_ns(G) < kCutSavingNs) ? cand : G;
}

struct SchedShared {
    int warp_sums[32];
    int b0;         // sequence that contains the first tile of this block's run
    int p0;         // global index of that sequence's first tile
    long long g0, g1;   // this block's run of tiles [g0, g1)
    int G;              // blocks that share the tiles (the launch's block count unless the plan is adaptive)
    int pair;           // uniform batch run on exactly two blocks per sequence (halves), see uniform_ctas
};

// Block-wide: total tile count T, and (b0, p0) for the tile `g0 = span_begin(cta)`.
// Every thread returns T; sh.b0/sh.p0 are valid after the call when the run is non-empty.
template <int NTHREADS>
__device__ inline int schedule_prologue(const LenView lengths, int B, int Lmax,
                                        int tile_shift, int G, int cta, SchedShared& sh, bool adaptive = false)
{
    const int tid = threadIdx.x;
    const int tile_rows = 1 << tile_shift;
    const int per = (B + NTHREADS - 1) / NTHREADS;
    const int b_lo = min(B, tid * per), b_hi = min(B, b_lo + per);
    int local = 0;
    const int nt_first = adaptive ? (clamp_len(lengths[0], Lmax) + tile_rows - 1) >> tile_shift : 0;
    bool uniform = adaptive;
    for (int b = b_lo; b < b_hi; ++b) {
        const int nt = (clamp_len(lengths[b], Lmax) + tile_rows - 1) >> tile_shift;
        local += nt;
        uniform = uniform && nt == nt_first;
    }
    // inclusive scan within the warp
    int incl = local;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) sh.warp_sums[warp] = incl;
    uniform = __syncthreads_and(uniform) != 0;
    // every thread adds up the warp totals itself (one barrier and one serial step less than a second scan)
    int T = 0, warp_offset = 0;
#pragma unroll
    for (int w = 0; w < NTHREADS / 32; ++w) {
        const int s = sh.warp_sums[w];
        T += s;
        if (w < warp) warp_offset += s;
    }
    if (uniform) G = uniform_ctas(B, nt_first, G);    // identical in every thread of every block
    if (tid == 0) { sh.G = G; sh.pair = (uniform && G == 2 * B && (nt_first & 1) == 0) ? 1 : 0; }
    int prefix = warp_offset + incl - local;          // tiles before this thread's first sequence
    if (T > 0 && cta < G) {
        const long long g0 = span_begin(cta, T, G);
        if (tid == 0) { sh.g0 = g0; sh.g1 = span_begin(cta + 1, T, G); }
        for (int b = b_lo; b < b_hi; ++b) {
            const int nt = (clamp_len(lengths[b], Lmax) + tile_rows - 1) >> tile_shift;
            if (nt > 0 && (long long)prefix <= g0 && g0 < (long long)prefix + nt) { sh.b0 = b; sh.p0 = prefix; }
            prefix += nt;
        }
    } else if (tid == 0) {
        sh.g0 = sh.g1 = 0;                            // a block beyond the chosen count owns no tiles
    }
    __syncthreads();
    return T;
}

// Walks the segments of one block's run.  All threads that use it hold identical state.
struct SegmentWalker {
    LenView lengths;
    int Lmax, tile_shift, B;
    long long g0, g1;     // this block's run
    long long g;          // next tile to hand out
    int b, len, nt;       // current sequence
    long long P;          // global index of its first tile

    __host__ __device__ void init(const LenView lengths_, int B_, int Lmax_, int tile_shift_, int T, int G,
                         int cta, int b0, int p0)
    {
        init_span(lengths_, B_, Lmax_, tile_shift_, span_begin(cta, T, G), span_begin(cta + 1, T, G), b0, p0);
    }
    // The same with the run [g0, g1) already known (the schedule prologue leaves it in shared memory).
    __host__ __device__ void init_span(const LenView lengths_, int B_, int Lmax_, int tile_shift_,
                                       long long g0_, long long g1_, int b0, int p0)
    {
        lengths = lengths_; B = B_; Lmax = Lmax_; tile_shift = tile_shift_;
        g0 = g0_; g1 = g1_; g = g0;
        if (g0 < g1) {
            b = b0; P = p0;
            len = clamp_len(lengths[b], Lmax);
            nt = (len + (1 << tile_shift) - 1) >> tile_shift;
        }
    }
    __host__ __device__ bool done() const { return g >= g1; }
    // Current segment: tiles [seg_t0, seg_t1) of sequence b (indices within the sequence).
    __host__ __device__ int seg_t0() const { return (int)(g - P); }
    __host__ __device__ int seg_t1() const { return (int)((g1 < P + nt ? g1 : P + nt) - P); }
    __host__ __device__ bool seg_is_whole() const { return g == P && g1 >= P + nt; }
    __host__ __device__ bool seg_owns_first_tile() const { return g == P; }
    __host__ __device__ int seg_slot(int cta) const { return (P <= g0) ? 2 * cta : 2 * cta + 1; }
    __host__ __device__ void next() {
        g = (g1 < P + nt) ? g1 : P + nt;
        if (g < g1) {
            P += nt;
            do {
                ++b;
                len = clamp_len(lengths[b], Lmax);
                nt = (len + (1 << tile_shift) - 1) >> tile_shift;
            } while (nt == 0 && b + 1 < B);
        }
    }
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Launchers (defined in their own translation units).
cudaError_t launch_fma(const Params& p, cudaStream_t stream);
cudaError_t launch_combine(const Params& p, cudaStream_t stream);
cudaError_t launch_tc(const Params& p, cudaStream_t stream);
cudaError_t launch_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int32_t* lengths,
                          int B, int D, int Lmax, unsigned char* workspace, cudaStream_t stream);
bool tc_supported(int H, int D);

}  // namespace mqa
