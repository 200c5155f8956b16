// Host side of the C ABI declared in include/mqa_decode.h: argument checks,
// the plan heuristic, and kernel launches.  No device memory is allocated here.
#include "../../include/mqa_decode.h"
#include "mqa_common.cuh"

#include <cstring>

namespace {

thread_local int g_last_launches = 0;

bool shape_ok(int B, int H, int D, int Lmax)
{
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) return false;
    if (!(D == 64 || D == 128 || D == 256)) return false;
    if (H > mqa::kMaxHeads) return false;
    const long long tiles = (long long)B * ((Lmax + 63) / 64);
    return tiles < (1ll << 31);
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int sm_count_or_default()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        cudaGetLastError();
        return 148;
    }
    return sms;
}

int tile_shift_of(int tile_rows) { return tile_rows == 64 ? 6 : tile_rows == 128 ? 7 : -1; }

}  // namespace

extern "C" {

const char* mqa_status_string(int status)
{
    switch (status) {
        case MQA_OK: return "ok";
        case MQA_ERR_INVALID_ARG: return "invalid argument";
        case MQA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case MQA_ERR_MISALIGNED: return "pointer not sufficiently aligned";
        case MQA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MQA_ERR_ARCH: return "device is not compute capability 10.x";
        case MQA_ERR_CUDA: return "CUDA call failed";
        case MQA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case MQA_ERR_CACHE_FULL: return "a sequence's cache had no free row for the appended token";
        default: return "unknown status";
    }
}

size_t mqa_decode_workspace_bytes(int B, int H, int D, int Lmax)
{
    if (!shape_ok(B, H, D, Lmax)) return 0;
    return mqa::workspace_bytes(B, H, D);
}

int mqa_workspace_init(void* workspace, size_t workspace_bytes, void* stream)
{
    if (!workspace) return MQA_ERR_INVALID_ARG;
    if (workspace_bytes < (size_t)mqa::kHeaderBytes) return MQA_ERR_WORKSPACE_TOO_SMALL;
    const size_t n = workspace_bytes;   // header, per-sequence records and arrival counters must start at zero
    if (cudaMemsetAsync(workspace, 0, n, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return MQA_ERR_CUDA;
    return MQA_OK;
}

int mqa_decode_plan(int B, int H, int D, int Lmax, int requested_path, mqa_plan_t* plan)
{
    if (!plan) return MQA_ERR_INVALID_ARG;
    if (!shape_ok(B, H, D, Lmax)) return (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) ? MQA_ERR_INVALID_ARG
                                                                                  : MQA_ERR_UNSUPPORTED_SHAPE;
    if (requested_path != MQA_PATH_AUTO && requested_path != MQA_PATH_FMA && requested_path != MQA_PATH_TC)
        return MQA_ERR_INVALID_ARG;
    const int sms = sm_count_or_default();
    int path = requested_path;
    if (path == MQA_PATH_TC && !mqa::tc_supported(H, D)) return MQA_ERR_UNSUPPORTED_SHAPE;
    if (path == MQA_PATH_AUTO) path = mqa::tc_supported(H, D) ? MQA_PATH_TC : MQA_PATH_FMA;
    plan->path = path;
    plan->tile_rows = (path == MQA_PATH_TC) ? 128 : 64;
    // An upper bound on the tile count (the host never reads `lengths`).
    const long long max_tiles = (long long)B * ((Lmax + plan->tile_rows - 1) / plan->tile_rows);
    // TC: one persistent block per SM (its shared-memory ring fills the SM).
    // FMA: two blocks per SM hide each other's tile-load latency.
    long long ctas = (path == MQA_PATH_TC) ? sms : 2ll * sms;
    if (ctas > max_tiles) ctas = max_tiles;
    if (ctas > MQA_MAX_CTAS) ctas = MQA_MAX_CTAS;
    if (ctas < 1) ctas = 1;
    plan->num_ctas = (int)ctas;
    plan->adaptive = (path == MQA_PATH_TC) ? 1 : 0;
    return MQA_OK;
}

// Scattered output of mqa_decode_scatter (out is null then).
struct ScatterArgs {
    float* const* dst;   // host array of n_dst device pointers
    int n_dst, b_offset, B_total;
};

static int decode_impl(const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* lengths, float* out,
                       int B, int H, int D, int Lmax, float scale,
                       const mqa_plan_t* plan,
                       void* workspace, size_t workspace_bytes, void* stream, void* event_after_split,
                       int kv_groups = 1, const ScatterArgs* scatter = nullptr)
{
    if (!q || !k_cache || !v_cache || !lengths || (!out && !scatter) || !workspace || !plan) return MQA_ERR_INVALID_ARG;
    if (scatter) {
        if (!scatter->dst || scatter->n_dst < 1 || scatter->n_dst > mqa::kMaxDst || scatter->b_offset < 0 ||
            scatter->B_total < 1)
            return MQA_ERR_INVALID_ARG;
        if (H % scatter->n_dst != 0 || (long long)scatter->b_offset + B > scatter->B_total) return MQA_ERR_INVALID_ARG;
        if (plan->path != MQA_PATH_TC) return MQA_ERR_UNSUPPORTED_SHAPE;   // only the tensor-core kernel scatters
        for (int r = 0; r < scatter->n_dst; ++r)
            if (!scatter->dst[r] || !aligned(scatter->dst[r], 16)) return scatter->dst[r] ? MQA_ERR_MISALIGNED : MQA_ERR_INVALID_ARG;
    }
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) return MQA_ERR_INVALID_ARG;
    if (!shape_ok(B, H, D, Lmax)) return MQA_ERR_UNSUPPORTED_SHAPE;
    if (!(scale == scale)) return MQA_ERR_INVALID_ARG;
    if (plan->num_ctas < 1 || plan->num_ctas > MQA_MAX_CTAS) return MQA_ERR_INVALID_ARG;
    if (plan->path != MQA_PATH_FMA && plan->path != MQA_PATH_TC) return MQA_ERR_INVALID_ARG;
    if (plan->tile_rows != ((plan->path == MQA_PATH_TC) ? 128 : 64)) return MQA_ERR_INVALID_ARG;
    if (plan->adaptive != 0 && plan->adaptive != 1) return MQA_ERR_INVALID_ARG;
    if (plan->path == MQA_PATH_TC && !mqa::tc_supported(H, D)) return MQA_ERR_UNSUPPORTED_SHAPE;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || (out && !aligned(out, 16)) ||
        !aligned(lengths, 4) || !aligned(workspace, 256))
        return MQA_ERR_MISALIGNED;
    if (workspace_bytes < mqa::workspace_bytes(B, H, D)) return MQA_ERR_WORKSPACE_TOO_SMALL;

    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    if (major != 10) return MQA_ERR_ARCH;

    mqa::Params p;
    p.q = static_cast<const uint16_t*>(q);
    p.k = static_cast<const uint16_t*>(k_cache);
    p.v = static_cast<const uint16_t*>(v_cache);
    p.lengths = mqa::LenView{lengths, kv_groups};
    p.out = out;
    p.n_dst = 0; p.b_offset = 0;
    for (int r = 0; r < mqa::kMaxDst; ++r) p.out_dst[r] = nullptr;
    if (scatter) {
        p.n_dst = scatter->n_dst; p.b_offset = scatter->b_offset;
        for (int r = 0; r < scatter->n_dst; ++r) p.out_dst[r] = scatter->dst[r];
    }
    p.B = B; p.H = H; p.D = D; p.Lmax = Lmax;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.tile_shift = tile_shift_of(plan->tile_rows);
    p.num_ctas = plan->num_ctas;
    p.adaptive = (plan->path == MQA_PATH_TC) ? plan->adaptive : 0;
    p.cluster = 1;
    // The tensor-core kernel's blocks wait for one another (merge of cut sequences), so all of them must be
    // resident at once: one block per SM at most.
    if (plan->path == MQA_PATH_TC && p.num_ctas > sm_count_or_default()) p.num_ctas = sm_count_or_default();
    p.lo_max_len = 0x7fffffff;
    p.workspace = static_cast<unsigned char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    cudaError_t e = (plan->path == MQA_PATH_TC) ? mqa::launch_tc(p, st) : mqa::launch_fma(p, st);
    if (e != cudaSuccess) return MQA_ERR_CUDA;
    if (event_after_split && cudaEventRecord(static_cast<cudaEvent_t>(event_after_split), st) != cudaSuccess)
        return MQA_ERR_CUDA;
    g_last_launches = 1;
    if (plan->path != MQA_PATH_TC) {   // the tensor-core kernel merges cut sequences itself
        e = mqa::launch_combine(p, st);
        if (e != cudaSuccess) return MQA_ERR_CUDA;
        g_last_launches = 2;
    }
    return MQA_OK;
}

int mqa_decode_with_plan(const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* lengths, float* out,
                         int B, int H, int D, int Lmax, float scale,
                         const mqa_plan_t* plan,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    return decode_impl(q, k_cache, v_cache, lengths, out, B, H, D, Lmax, scale, plan,
                       workspace, workspace_bytes, stream, nullptr);
}

int mqa_decode_profiled(const void* q, const void* k_cache, const void* v_cache,
                        const int32_t* lengths, float* out,
                        int B, int H, int D, int Lmax, float scale,
                        const mqa_plan_t* plan,
                        void* workspace, size_t workspace_bytes, void* stream, void* event_after_split)
{
    mqa_plan_t local;
    if (!plan) {
        const int rc = mqa_decode_plan(B, H, D, Lmax, MQA_PATH_AUTO, &local);
        if (rc != MQA_OK) return rc;
        plan = &local;
    }
    return decode_impl(q, k_cache, v_cache, lengths, out, B, H, D, Lmax, scale, plan,
                       workspace, workspace_bytes, stream, event_after_split);
}

int mqa_decode(const void* q, const void* k_cache, const void* v_cache,
               const int32_t* lengths, float* out,
               int B, int H, int D, int Lmax, float scale,
               void* workspace, size_t workspace_bytes, void* stream)
{
    mqa_plan_t plan;
    const int rc = mqa_decode_plan(B, H, D, Lmax, MQA_PATH_AUTO, &plan);
    if (rc != MQA_OK) return rc;
    return mqa_decode_with_plan(q, k_cache, v_cache, lengths, out, B, H, D, Lmax, scale, &plan,
                                workspace, workspace_bytes, stream);
}

int mqa_decode_scatter(const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* lengths, float* const* out_dst, int n_dst, int b_offset, int B_total,
                       int B, int H, int D, int Lmax, float scale,
                       void* workspace, size_t workspace_bytes, void* stream)
{
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) return MQA_ERR_INVALID_ARG;
    mqa_plan_t plan;
    const int rc = mqa_decode_plan(B, H, D, Lmax, MQA_PATH_TC, &plan);
    if (rc != MQA_OK) return rc;
    ScatterArgs sc{out_dst, n_dst, b_offset, B_total};
    return decode_impl(q, k_cache, v_cache, lengths, nullptr, B, H, D, Lmax, scale, &plan,
                       workspace, workspace_bytes, stream, nullptr, 1, &sc);
}

int mqa_append_decode(const void* q, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache, int32_t* lengths, float* out,
                      int B, int H, int D, int Lmax, float scale,
                      void* workspace, size_t workspace_bytes, void* stream)
{
    if (!q || !k_new || !v_new || !k_cache || !v_cache || !lengths || !out || !workspace) return MQA_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) return MQA_ERR_INVALID_ARG;
    if (!shape_ok(B, H, D, Lmax)) return MQA_ERR_UNSUPPORTED_SHAPE;
    if (!(scale == scale)) return MQA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) ||
        !aligned(out, 16) || !aligned(lengths, 4) || !aligned(workspace, 256))
        return MQA_ERR_MISALIGNED;
    if (workspace_bytes < mqa::workspace_bytes(B, H, D)) return MQA_ERR_WORKSPACE_TOO_SMALL;
    mqa_plan_t plan;
    int rc = mqa_decode_plan(B, H, D, Lmax, MQA_PATH_AUTO, &plan);
    if (rc != MQA_OK) return rc;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    if (major != 10) return MQA_ERR_ARCH;
    if (mqa::launch_append(k_new, v_new, k_cache, v_cache, lengths, B, D, Lmax,
                           static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return MQA_ERR_CUDA;
    rc = decode_impl(q, k_cache, v_cache, lengths, out, B, H, D, Lmax, scale, &plan, workspace, workspace_bytes,
                     stream, nullptr);
    if (rc == MQA_OK) g_last_launches += 1;
    return rc;
}

int mqa_decode_grouped(const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* lengths, float* out,
                       int B, int H, int KVH, int D, int Lmax, float scale,
                       void* workspace, size_t workspace_bytes, void* stream)
{
    if (KVH <= 0 || H <= 0 || B <= 0) return MQA_ERR_INVALID_ARG;
    if (H % KVH != 0) return MQA_ERR_UNSUPPORTED_SHAPE;
    if ((long long)B * KVH >= (1ll << 31)) return MQA_ERR_UNSUPPORTED_SHAPE;
    // Each (sequence, key/value head) pair is one multiquery problem: H/KVH query heads sharing one K/V head
    // over rows [0, lengths[b]).  With the caches laid out [B, KVH, Lmax, D] and q/out as [B, H, D] (the heads
    // of a group adjacent) that is mqa_decode on B*KVH sequences, the lengths read through a grouped view.
    const int Bg = B * KVH, Hg = H / KVH;
    mqa_plan_t plan;
    const int rc = mqa_decode_plan(Bg, Hg, D, Lmax, MQA_PATH_AUTO, &plan);
    if (rc != MQA_OK) return rc;
    return decode_impl(q, k_cache, v_cache, lengths, out, Bg, Hg, D, Lmax, scale, &plan,
                       workspace, workspace_bytes, stream, nullptr, KVH);
}

size_t mqa_decode_grouped_workspace_bytes(int B, int H, int KVH, int D, int Lmax)
{
    if (KVH <= 0 || H <= 0 || B <= 0 || H % KVH != 0 || (long long)B * KVH >= (1ll << 31)) return 0;
    return mqa_decode_workspace_bytes(B * KVH, H / KVH, D, Lmax);
}

int mqa_check_status(void* workspace, void* stream)
{
    if (!workspace) return MQA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int status = 0;
    if (cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MQA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MQA_ERR_CUDA;
    if (status != 0) {
        if (cudaMemsetAsync(workspace, 0, sizeof(int), st) != cudaSuccess) return MQA_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return MQA_ERR_CUDA;
    }
    return status;
}

static size_t up256(size_t x) { return (x + 255) / 256 * 256; }

size_t mqa_decode_host_scratch_bytes(int B, int H, int D, int Lmax)
{
    if (!shape_ok(B, H, D, Lmax)) return 0;
    const size_t qb = up256((size_t)B * H * D * 2), kb = up256((size_t)B * Lmax * D * 2);
    const size_t lb = up256((size_t)B * 4), ob = up256((size_t)B * H * D * 4);
    return qb + 2 * kb + lb + ob + up256(mqa::workspace_bytes(B, H, D));
}

int mqa_decode_host(const void* q_host, const void* k_cache_host, const void* v_cache_host,
                    const int32_t* lengths_host, float* out_host,
                    int B, int H, int D, int Lmax, float scale,
                    void* scratch, size_t scratch_bytes, void* stream)
{
    if (!q_host || !k_cache_host || !v_cache_host || !lengths_host || !out_host || !scratch) return MQA_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || D <= 0 || Lmax <= 0) return MQA_ERR_INVALID_ARG;
    if (!shape_ok(B, H, D, Lmax)) return MQA_ERR_UNSUPPORTED_SHAPE;
    if (!aligned(scratch, 256)) return MQA_ERR_MISALIGNED;
    if (scratch_bytes < mqa_decode_host_scratch_bytes(B, H, D, Lmax)) return MQA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qn = (size_t)B * H * D * 2, kn = (size_t)B * Lmax * D * 2, ln = (size_t)B * 4, on = (size_t)B * H * D * 4;
    unsigned char* base = static_cast<unsigned char*>(scratch);
    unsigned char* dq = base;
    unsigned char* dk = dq + up256(qn);
    unsigned char* dv = dk + up256(kn);
    unsigned char* dl = dv + up256(kn);
    unsigned char* dout = dl + up256(ln);
    unsigned char* dws = dout + up256(on);
    const size_t wsn = mqa::workspace_bytes(B, H, D);
    if (cudaMemcpyAsync(dq, q_host, qn, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dk, k_cache_host, kn, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dv, v_cache_host, kn, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dl, lengths_host, ln, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return MQA_ERR_CUDA;
    int rc = mqa_workspace_init(dws, wsn, stream);
    if (rc != MQA_OK) return rc;
    rc = mqa_decode(dq, dk, dv, reinterpret_cast<const int32_t*>(dl), reinterpret_cast<float*>(dout),
                    B, H, D, Lmax, scale, dws, wsn, stream);
    if (rc != MQA_OK) return rc;
    if (cudaMemcpyAsync(out_host, dout, on, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MQA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MQA_ERR_CUDA;
    return MQA_OK;
}

int mqa_last_launch_count(void) { return g_last_launches; }

int mqa_uniform_ctas(int B, int tiles_per_sequence, int num_ctas)
{
    if (B <= 0 || tiles_per_sequence <= 0 || num_ctas <= 0 || num_ctas > MQA_MAX_CTAS) return -MQA_ERR_INVALID_ARG;
    return mqa::uniform_ctas(B, tiles_per_sequence, num_ctas);
}

int mqa_debug_schedule(const int32_t* lengths_host, int B, int Lmax, int tile_rows, int num_ctas, int cta,
                       int32_t* records, int max_segments)
{
    if (!lengths_host || !records || B <= 0 || Lmax <= 0 || max_segments < 0) return -MQA_ERR_INVALID_ARG;
    const int shift = tile_shift_of(tile_rows);
    if (shift < 0 || num_ctas < 1 || num_ctas > MQA_MAX_CTAS || cta < 0 || cta >= num_ctas) return -MQA_ERR_INVALID_ARG;
    // Host replay of the device prologue: total tile count and the sequence holding the run's first tile.
    long long T = 0;
    for (int b = 0; b < B; ++b) T += (mqa::clamp_len(lengths_host[b], Lmax) + tile_rows - 1) >> shift;
    if (T >= (1ll << 31)) return -MQA_ERR_UNSUPPORTED_SHAPE;
    if (T == 0) return 0;
    const long long g0 = mqa::span_begin(cta, (int)T, num_ctas);
    int b0 = 0, p0 = 0;
    long long prefix = 0;
    for (int b = 0; b < B; ++b) {
        const int nt = (mqa::clamp_len(lengths_host[b], Lmax) + tile_rows - 1) >> shift;
        if (nt > 0 && prefix <= g0 && g0 < prefix + nt) { b0 = b; p0 = (int)prefix; }
        prefix += nt;
    }
    mqa::SegmentWalker w;
    w.init(mqa::LenView{lengths_host, 1}, B, Lmax, shift, (int)T, num_ctas, cta, b0, p0);
    int n = 0;
    for (; !w.done(); w.next()) {
        if (n < max_segments) {
            int32_t* r = records + 7 * n;
            r[0] = w.b; r[1] = w.seg_t0(); r[2] = w.seg_t1(); r[3] = w.seg_is_whole() ? 1 : 0;
            r[4] = w.seg_is_whole() ? -1 : w.seg_slot(cta);
            r[5] = w.seg_owns_first_tile() ? 1 : 0;
            r[6] = mqa::cta_of_tile(w.P + w.nt - 1, (int)T, num_ctas);
        }
        ++n;
    }
    return n;
}

}  // extern "C"
