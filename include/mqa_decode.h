/*
 * mqa_decode.h - C ABI of the B200 (sm_100a) multiquery decode-attention library.
 *
 * Operation ("Efficiently Scaling Transformer Inference", Section 3.3): in
 * multiquery attention every sequence has n_heads query heads but a single key
 * head and a single value head that all query heads share.  In the generate
 * phase there is one query token per sequence, attending to that sequence's
 * whole KV cache; the step's cost is reading the cache from HBM once
 * (Section 2, "Memory costs"; Section 2.1).  For every sequence b and head h:
 *
 *     out[b,h,:] = sum_{l < lengths[b]} softmax_l( scale * q[b,h,:].k[b,l,:] ) * v[b,l,:]
 *
 * The kernels read each K/V tile once and use it for all H heads, evaluate the
 * softmax in base 2 (Section 3.5 names base-2 softmax as an implementation
 * choice; the function is the same), split the sequence axis across thread
 * blocks with running-max partial results, and merge the partials with a
 * log-sum-exp combine.
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer unless the parameter name ends in _host.
 *   - Layouts are row-major and dense: q [B,H,D], k_cache/v_cache [B,Lmax,D],
 *     out [B,H,D], lengths [B].  q/k/v are bf16, out is fp32, lengths int32.
 *   - The caller owns every buffer.  The library allocates no device memory.
 *   - Calls enqueue work on `stream` and return without synchronising, except
 *     mqa_check_status and mqa_decode_host, which synchronise the stream.
 *   - Inputs are read-only.  out is fully overwritten for every (b,h).
 *   - lengths[b] counts the valid cache rows of sequence b (the current token's
 *     K/V row already appended) and is clamped into [0, Lmax] on the device.
 *     lengths[b] == 0 gives an all-zero output row.  Cache rows at or beyond
 *     lengths[b] may hold any bits (NaN included); they never affect out.
 *   - Every function that returns int returns an mqa_status_t.  On any error
 *     nothing is launched.
 *   - Same inputs and same plan give bit-identical output.
 *   - Accuracy (tensor-core path): probabilities enter the weighted-value product as bf16; sequences of
 *     up to 1024 rows also carry the low-order bf16 half (about 16 bits in all).  On N(0,1) inputs the
 *     error stays below 0.3x of 2e-3*(1+|ref|).  The environment variable MQA_LO_MAX_LEN moves the
 *     length limit (2147483647 = always both halves).
 *   - Thread safety: concurrent calls are safe when they use different
 *     workspaces.  Two calls sharing a workspace must be stream-ordered.
 *   - Launches: the tensor-core path is ONE cooperative launch per call (its blocks wait for one another when
 *     they merge a sequence that was cut, so all of them must be resident: at most one block per SM, and two
 *     such calls on different streams run one after the other).  For some uniform batches the launch uses
 *     thread-block clusters of two (environment variable MQA_NO_CLUSTER turns that off).  The launch can be
 *     captured in a CUDA graph.  The FMA path enqueues two ordinary kernels.
 */
#ifndef MQA_DECODE_H_
#define MQA_DECODE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MQA_OK = 0,
    MQA_ERR_INVALID_ARG = 1,         /* null pointer, non-positive size, bad plan field   */
    MQA_ERR_UNSUPPORTED_SHAPE = 2,   /* D not in {64,128,256}, H > 64, tile count overflow */
    MQA_ERR_MISALIGNED = 3,          /* q/k/v/out/workspace not 16-byte aligned            */
    MQA_ERR_WORKSPACE_TOO_SMALL = 4,
    MQA_ERR_ARCH = 5,                /* current device is not compute capability 10.x      */
    MQA_ERR_CUDA = 6,                /* a CUDA runtime/driver call failed                  */
    MQA_ERR_TIMEOUT = 7,             /* a bounded device-side wait ran out (see check_status) */
    MQA_ERR_CACHE_FULL = 8           /* mqa_append_decode: some sequence had no free cache row (see check_status) */
} mqa_status_t;

/* Kernel families (mqa_plan_t.path). */
enum {
    MQA_PATH_AUTO = 0,
    MQA_PATH_FMA = 1,   /* fp32 FMA kernel, any supported shape                      */
    MQA_PATH_TC = 2     /* tcgen05 tensor-core kernel with TMA staging: D in {128,256}          */
};

/*
 * Execution plan: which kernel family, how many persistent thread blocks share
 * the flattened list of K/V tiles, and the tile height in cache rows.  The
 * sequence axis is split wherever a block's share of tiles ends, so the split
 * count per sequence follows from (B, lengths, num_ctas).
 */
typedef struct {
    int path;        /* MQA_PATH_FMA or MQA_PATH_TC (AUTO only as a request)  */
    int num_ctas;    /* 1 .. MQA_MAX_CTAS; the TC path runs min(num_ctas, SM count) blocks
                        (its blocks wait for one another, so all must be resident) */
    int tile_rows;   /* cache rows per tile: 64 (FMA) or 128 (TC)              */
    int adaptive;    /* TC path, 0 or 1: when every sequence of the batch owns the same
                        number of tiles the kernel may share them among fewer blocks
                        (mqa_uniform_ctas) so that the cuts fall on sequence boundaries;
                        mqa_decode_plan sets it, 0 pins the block count to num_ctas */
} mqa_plan_t;

#define MQA_MAX_CTAS 592          /* upper bound on mqa_plan_t.num_ctas (4 per SM on 148 SMs) */
#define MQA_MAX_HEADS 64

/* Human-readable name of a status code (static storage, never NULL). */
const char* mqa_status_string(int status);

/*
 * Bytes of device workspace mqa_decode needs for this shape under ANY plan the
 * library may choose: a 256-byte header (device status word, tile total), one
 * 8-byte record and one 4-byte arrival counter per sequence (each array rounded
 * up to 256 bytes), and two partial-result slots per thread block
 * (per slot: running max and running sum per head, and the unnormalised fp32
 * accumulator [H,D]).  Returns 0 for an unsupported shape.  Host-only; no
 * device is touched.
 */
size_t mqa_decode_workspace_bytes(int B, int H, int D, int Lmax);

/*
 * Zero the workspace (device status word, per-sequence records and arrival
 * counters must start at zero; the kernels leave them zero again).  Call once
 * after allocating the workspace, before the first mqa_decode that uses it,
 * and again after a call that reported MQA_ERR_TIMEOUT.
 */
int mqa_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * The heuristic's plan for a shape on the current device (reads the SM count;
 * falls back to 148 if no device is present).  Host-only otherwise.
 * `requested_path` is MQA_PATH_AUTO, MQA_PATH_FMA or MQA_PATH_TC; a path the
 * shape does not support gives MQA_ERR_UNSUPPORTED_SHAPE.
 */
int mqa_decode_plan(int B, int H, int D, int Lmax, int requested_path, mqa_plan_t* plan);

/*
 * One decode-attention step (Section 3.3; formula at the top of this file).
 *   q          device bf16  [B,H,D]      16-byte aligned
 *   k_cache    device bf16  [B,Lmax,D]   16-byte aligned
 *   v_cache    device bf16  [B,Lmax,D]   16-byte aligned
 *   lengths    device int32 [B]          read on the device only
 *   out        device fp32  [B,H,D]      16-byte aligned, overwritten
 *   scale      multiplies the fp32 logit (not folded into q)
 *   workspace  device, 256-byte aligned, >= mqa_decode_workspace_bytes(...)
 *   stream     cudaStream_t (NULL = legacy default stream)
 * Supported: D in {64,128,256}; 1 <= H <= 64; B, Lmax >= 1 with
 * B*ceil(Lmax/64) < 2^31.
 */
int mqa_decode(const void* q, const void* k_cache, const void* v_cache,
               const int32_t* lengths, float* out,
               int B, int H, int D, int Lmax, float scale,
               void* workspace, size_t workspace_bytes, void* stream);

/*
 * One whole generate step of the attention layer (Section 2.2: every decode step yields one new token
 * per sequence whose key/value joins the cache; Section 3.3: that step has one token of Q, K, V per
 * sequence against a cache of many): append, then attend.
 *   k_new, v_new  device bf16 [B,D]   this step's key and value row of every sequence, 16-byte aligned
 *   k_cache, v_cache                  device bf16 [B,Lmax,D], WRITTEN: row lengths[b] of sequence b
 *   lengths       device int32 [B]    in: valid rows before the step; out: incremented by one
 * For every b with 0 <= lengths[b] < Lmax the new rows are stored at index lengths[b] and lengths[b]
 * grows by one; then out is computed exactly as by mqa_decode over the lengthened cache.  A sequence
 * with lengths[b] >= Lmax (or negative) gets nothing appended, keeps its length, is attended over its
 * clamped old length, and MQA_ERR_CACHE_FULL is recorded in the workspace status word (read it with
 * mqa_check_status).  Two kernels are enqueued (append, split); other arguments as in mqa_decode.
 */
int mqa_append_decode(const void* q, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache, int32_t* lengths, float* out,
                      int B, int H, int D, int Lmax, float scale,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Batch-sharded decode attention with the output already laid out for a heads-sharded consumer
 * (Section 3.3: multiquery attention is sharded over the batch, at the price of an all-to-all that moves
 * the per-token tensors between the heads-sharded and the batch-sharded layout; Figure 5).  This call is one
 * rank's attention over its slice of the batch, fused with the all-to-all of the OUTPUT: instead of one
 * [B,H,D] array, head h of local sequence b is stored to
 *     out_dst[h / (H/n_dst)] + ((b_offset + b) * (H/n_dst) + h % (H/n_dst)) * D,
 * i.e. into row b_offset + b of destination rank r's [B_total, H/n_dst, D] fp32 buffer.  The destinations are
 * plain device pointers: this GPU's own memory, or peers' memory mapped into this process (peer access /
 * symmetric memory over NVLink); the kernel reaches them with ordinary stores, never with TMA multicast.
 *   out_dst   HOST array of n_dst device pointers (copied into the launch), each 16-byte aligned, each a
 *             buffer of at least B_total * (H/n_dst) * D floats; rows outside [b_offset, b_offset + B) are
 *             not touched
 *   n_dst     1..16, a divisor of H;   b_offset >= 0, b_offset + B <= B_total
 * The caller synchronises the ranks before the consumer reads (the stores are complete when the stream
 * reaches the end of this call's kernel).  Tensor-core path only (D in {128, 256}): other shapes return
 * MQA_ERR_UNSUPPORTED_SHAPE.  Everything else as mqa_decode.
 */
int mqa_decode_scatter(const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* lengths, float* const* out_dst, int n_dst, int b_offset, int B_total,
                       int B, int H, int D, int Lmax, float scale,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Decode attention with KVH key/value heads per sequence (grouped-query attention; KVH == H is the
 * multihead attention the paper compares against in Section 4.2 and Table 1, KVH == 1 is mqa_decode).
 * Query head h uses key/value head h / (H/KVH).  The cache then holds KVH times the bytes, which is the
 * memory-time cost Section 3.3 attributes to multihead attention.
 *   q        device bf16 [B,H,D]            the H/KVH heads of one group adjacent
 *   k_cache  device bf16 [B,KVH,Lmax,D]     (one contiguous [Lmax,D] cache per key/value head)
 *   v_cache  device bf16 [B,KVH,Lmax,D]
 *   lengths  device int32 [B]               shared by the KVH heads of a sequence
 *   out      device fp32 [B,H,D]
 *   workspace  >= mqa_decode_grouped_workspace_bytes(B, H, KVH, D, Lmax), 256-byte aligned, initialised
 * H must be a multiple of KVH; H/KVH and D obey the limits of mqa_decode.  Everything else as mqa_decode.
 */
int mqa_decode_grouped(const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* lengths, float* out,
                       int B, int H, int KVH, int D, int Lmax, float scale,
                       void* workspace, size_t workspace_bytes, void* stream);
size_t mqa_decode_grouped_workspace_bytes(int B, int H, int KVH, int D, int Lmax);

/* Same as mqa_decode, with an explicit plan (tests and tuning). */
int mqa_decode_with_plan(const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* lengths, float* out,
                         int B, int H, int D, int Lmax, float scale,
                         const mqa_plan_t* plan,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * Same as mqa_decode_with_plan (plan == NULL selects the heuristic's plan), and
 * additionally records `event_after_split` (a cudaEvent_t; may be NULL) on the
 * stream between the split kernel and the combine kernel, so a benchmark can
 * time the bandwidth-bound kernel on its own.
 */
int mqa_decode_profiled(const void* q, const void* k_cache, const void* v_cache,
                        const int32_t* lengths, float* out,
                        int B, int H, int D, int Lmax, float scale,
                        const mqa_plan_t* plan,
                        void* workspace, size_t workspace_bytes, void* stream,
                        void* event_after_split);

/*
 * Synchronise `stream`, read the device status word from the workspace header,
 * reset it to zero and return it (MQA_OK; MQA_ERR_TIMEOUT if a bounded wait
 * inside a kernel gave up, the output of that call is then undefined;
 * MQA_ERR_CACHE_FULL after mqa_append_decode found a full cache).
 */
int mqa_check_status(void* workspace, void* stream);

/*
 * Device scratch needed by mqa_decode_host: room for q, both caches, lengths,
 * out (each rounded up to 256 bytes) plus mqa_decode_workspace_bytes.
 */
size_t mqa_decode_host_scratch_bytes(int B, int H, int D, int Lmax);

/*
 * End-to-end convenience call for HOST buffers (pinned memory recommended):
 * copies q/k/v/lengths into `scratch` (device memory supplied by the caller),
 * runs mqa_decode, copies out back to out_host and synchronises `stream`.
 * The scratch header is initialised by this call.
 */
int mqa_decode_host(const void* q_host, const void* k_cache_host, const void* v_cache_host,
                    const int32_t* lengths_host, float* out_host,
                    int B, int H, int D, int Lmax, float scale,
                    void* scratch, size_t scratch_bytes, void* stream);

/* Number of kernels the last successful mqa_decode* call on this host thread
 * launched (for launch accounting in benchmarks). */
int mqa_last_launch_count(void);

/*
 * Allocation-free variant of mqa_decode (the paper has no counterpart; this is
 * a packaging convenience of this library).  It is for callers that cannot
 * allocate device memory at all - code embedded in a host application that
 * owns every byte of the GPU, a serving loop that may not enter the allocator,
 * a sandbox where allocation calls are unavailable - and therefore cannot
 * supply the workspace mqa_decode asks for.  The workspace is instead a fixed
 * array of MQA_STATIC_WORKSPACE_BYTES inside the library's device image; every
 * GPU that loads the library holds that much memory until the process exits.
 *
 * Arguments, layouts and results are those of mqa_decode, without the
 * workspace.  Limits: the shape must fit the fixed array, i.e.
 *   256 + roundup(8*B, 256) + roundup(4*B, 256) + 2 * 4*(2*roundup(H,4) + H*D) <= MQA_STATIC_WORKSPACE_BYTES;
 * a larger shape returns MQA_ERR_WORKSPACE_TOO_SMALL and launches nothing.
 * When the heuristic's block count would not fit, fewer blocks are used.
 * The call makes no cudaMalloc/cudaFree and uses no allocating library
 * routine.  The first call on each device looks up the array's device address
 * (once per device, with that device current); make that first call outside of
 * any stream capture.
 *
 * All calls on one device share the array, and it keeps the last call's
 * contents: the call clears the part that must start at zero (header, records,
 * counters) on `stream` before launching.  Calls whose kernels may overlap on the GPU
 * (different streams without ordering) race on the array; order them.  A
 * time-out of a bounded device-side wait cannot be read back through this
 * entry point; use mqa_decode with mqa_check_status to diagnose one.
 */
#define MQA_STATIC_WORKSPACE_BYTES (20u << 20)
int mqa_decode_static(const void* q, const void* k_cache, const void* v_cache,
                      const int32_t* lengths, float* out,
                      int B, int H, int D, int Lmax, float scale, void* stream);

/*
 * Block count an adaptive plan uses for a batch in which each of the B sequences
 * owns `tiles_per_sequence` K/V tiles, given the plan's num_ctas: the split-count
 * heuristic for uniform batches (the paper fixes no split; Section 3.3 only
 * states that the K/V cache load dominates decode attention).  With an even
 * share of the flattened tiles almost every block boundary cuts a sequence, and
 * each cut costs two partial epilogues and a merge.  A block count that divides
 * B (whole sequences per block), or a multiple of B whose factor divides the
 * tile count (every sequence in equal parts), avoids that and is chosen when
 * the modelled slow-down of the K/V stream (fewer streaming SMs) stays below
 * the modelled saving.  Returns num_ctas itself when no such count qualifies.
 * Any other batch always runs on num_ctas blocks.  Host-only, no device is
 * touched; returns a negated mqa_status_t for non-positive arguments.
 */
int mqa_uniform_ctas(int B, int tiles_per_sequence, int num_ctas);

/*
 * Host replay of the device tile schedule, for tests and tooling (no device is
 * touched).  The K/V tiles of all sequences are numbered sequence-major and
 * block `cta` of `num_ctas` takes a contiguous run of them; each piece of a
 * sequence inside one run is a segment.  Writes up to max_segments records of
 * 7 int32 each: {sequence, first tile, end tile (exclusive, both within the
 * sequence), whole-sequence flag, partial slot (-1 if whole), owns-first-tile
 * flag, block that owns the sequence's last tile}.  lengths_host is a HOST
 * array.  Returns the number of segments of that block, or a negated
 * mqa_status_t.
 */
int mqa_debug_schedule(const int32_t* lengths_host, int B, int Lmax, int tile_rows, int num_ctas, int cta,
                       int32_t* records, int max_segments);

#ifdef __cplusplus
}
#endif
#endif /* MQA_DECODE_H_ */
