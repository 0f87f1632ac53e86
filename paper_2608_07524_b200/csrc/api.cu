// C ABI of libdcp: argument checks, tensor-map construction, workspace carving and kernel launches.
// Definitions of every operation are in include/dcp.h.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/dcp.h"
#include "attn_kernels.h"
#include "dcp_internal.h"
#include "sched.cuh"

namespace dcp {

char* error_buffer() {
    static thread_local char buf[512] = "";
    return buf;
}

namespace {

std::atomic<int64_t> g_launches{0};
std::atomic<int> g_input_order{0};      // dcp_set_work_order: 1 = list sequences as they come
std::atomic<int> g_short_path{1};       // dcp_set_short_sequence_path: 0 = batches of very short sequences run on the tile kernels

// Optional per-kernel timing: event pairs recorded on the caller's stream around every launch.  Events
// are created once and recycled through a pool (dcp_profile_read hands them back), so that a timed
// launch costs two event records and no create/destroy.
struct TimedLaunch {
    int kernel, device;
    cudaEvent_t start, stop;
};
constexpr int kMaxDevices = 64;
std::mutex g_prof_mu;
std::atomic<int> g_prof_on{0};
std::vector<TimedLaunch> g_prof_pending;
std::vector<cudaEvent_t> g_event_pool[kMaxDevices];      // an event belongs to the device it was created on

cudaEvent_t pool_take(int device) {
    {
        std::lock_guard<std::mutex> lock(g_prof_mu);
        std::vector<cudaEvent_t>& pool = g_event_pool[device];
        if (!pool.empty()) {
            cudaEvent_t e = pool.back();
            pool.pop_back();
            return e;
        }
    }
    cudaEvent_t e = nullptr;
    return cudaEventCreate(&e) == cudaSuccess ? e : nullptr;
}

struct ScopedTimer {
    int kernel, device = 0;
    cudaStream_t stream;
    cudaEvent_t start = nullptr, stop = nullptr;
    ScopedTimer(int k, cudaStream_t s) : kernel(k), stream(s) {
        if (!g_prof_on.load()) return;
        if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return;
        start = pool_take(device);
        stop = pool_take(device);
        if (!start || !stop) {
            std::lock_guard<std::mutex> lock(g_prof_mu);
            if (start) g_event_pool[device].push_back(start);
            if (stop) g_event_pool[device].push_back(stop);
            start = stop = nullptr;
            return;
        }
        cudaEventRecord(start, stream);
    }
    ~ScopedTimer() {
        if (!start) return;
        cudaEventRecord(stop, stream);
        std::lock_guard<std::mutex> lock(g_prof_mu);
        g_prof_pending.push_back({kernel, device, start, stop});
    }
};

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up at run time so that the library loads (and the planner
// works) on machines without a CUDA driver.
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0;
};

// Properties of the current device, cached per device id.
int device_info(DeviceInfo* out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(DCP_ERR_CUDA, "cudaGetDevice failed (no CUDA device?)");
    if (dev < 0 || dev >= 64) return fail(DCP_ERR_CUDA, "device index %d out of range", dev);
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev].device != dev) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return fail(DCP_ERR_CUDA, "cudaGetDeviceProperties failed");
        cache[dev].device = dev;
        cache[dev].sm_count = prop.multiProcessorCount;
        cache[dev].cc_major = prop.major;
    }
    *out = cache[dev];
    return DCP_OK;
}

// [T, H, d] bf16 viewed as a 3-D tensor (d, H, T); a box is 64 columns x 1 head x 128 tokens,
// written to shared memory as 128 rows of 128 bytes with the 128-byte swizzle.  Rows past T are
// zero-filled.  Consecutive tokens are row_stride elements apart (n_heads * head_dim when the tensor is
// contiguous; more when it is a group of heads inside a wider tensor).
int make_map(CUtensorMap* map, const void* base, int32_t total_tokens, int32_t n_heads, int32_t head_dim,
             int64_t row_stride) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return fail(DCP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the CUDA driver");
    const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_heads, (cuuint64_t)total_tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)row_stride * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)kTile};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                           elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(DCP_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return DCP_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(const char* fn, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen, int32_t n_heads,
                int32_t head_dim, float softmax_scale) {
    if (n_seqs < 0 || total_tokens < 0 || max_seqlen < 0 || n_heads < 1)
        return fail(DCP_ERR_INVALID_ARG, "%s: negative size or n_heads < 1", fn);
    if (n_seqs > 65535) return fail(DCP_ERR_UNSUPPORTED, "%s: at most 65535 sequences per call", fn);
    if (n_heads > 65535) return fail(DCP_ERR_UNSUPPORTED, "%s: at most 65535 heads", fn);
    if (head_dim < 8 || head_dim > 128 || head_dim % 8 != 0)
        return fail(DCP_ERR_UNSUPPORTED, "%s: head_dim %d is not supported (a multiple of 8 up to 128)", fn, head_dim);
    if (max_seqlen > total_tokens) return fail(DCP_ERR_INVALID_ARG, "%s: max_seqlen exceeds total_tokens", fn);
    if (!(softmax_scale >= 0.f) || std::isinf(softmax_scale))
        return fail(DCP_ERR_INVALID_ARG, "%s: softmax_scale must be finite and >= 0 (0 selects 1/sqrt(d))", fn);
    if ((int64_t)total_tokens * n_heads >= ((int64_t)1 << 31))
        return fail(DCP_ERR_UNSUPPORTED, "%s: total_tokens * n_heads must be below 2^31", fn);
    return DCP_OK;
}

int check_stride(const char* fn, int64_t token_stride, int32_t n_heads, int32_t head_dim) {
    if (token_stride < (int64_t)n_heads * head_dim || token_stride % 8 != 0)
        return fail(DCP_ERR_INVALID_ARG, "%s: token_stride must be a multiple of 8 elements and at least n_heads * head_dim", fn);
    if (token_stride >= ((int64_t)1 << 38)) return fail(DCP_ERR_UNSUPPORTED, "%s: token_stride too large", fn);
    return DCP_OK;
}

SchedView carve_sched(void* workspace, int32_t n_seqs) {
    SchedView s;
    uint8_t* base = static_cast<uint8_t*>(workspace);
    s.hdr = reinterpret_cast<WorkspaceHeader*>(base);
    s.spans = reinterpret_cast<CtaSpan*>(base + sizeof(WorkspaceHeader));
    base += sizeof(WorkspaceHeader) + kSpanBytes;
    s.order = reinterpret_cast<const int32_t*>(base);
    s.prefix = reinterpret_cast<const uint32_t*>(base + sizeof(int32_t) * (size_t)n_seqs);
    s.tile_prefix = s.prefix + (size_t)n_seqs + 1;
    s.vcu = reinterpret_cast<const int32_t*>(s.tile_prefix + (size_t)n_seqs + 1);
    s.n_seqs = n_seqs;
    return s;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Whether a call takes the path for batches of very short sequences (see attn_small.cu).
bool short_sequence_path(int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen) {
    return g_short_path.load() != 0 && small_path_fits(n_seqs, total_tokens, max_seqlen);
}

// Batches whose longest sequence has at most this many tokens (64 key tiles) run the forward variant for short items.
constexpr int32_t kShortItemMaxLen = 8192;

// The kernels work on 64 or 128 columns per head; other head dimensions run zero-padded to the next of the two.
size_t padded_dim(int32_t head_dim) { return head_dim <= 64 ? 64 : 128; }

}  // namespace
}  // namespace dcp

using namespace dcp;

extern "C" const char* dcp_last_error(void) { return error_buffer(); }

extern "C" int64_t dcp_launch_count(void) { return g_launches.load(); }

extern "C" int dcp_varlen_attn_workspace(int32_t total_tokens, int32_t n_seqs, int32_t n_heads, int32_t head_dim,
                                         size_t* fwd_bytes, size_t* bwd_bytes) {
    if (total_tokens < 0 || n_seqs < 0 || n_heads < 1 || head_dim < 1)
        return fail(DCP_ERR_INVALID_ARG, "dcp_varlen_attn_workspace: bad sizes");
    const size_t sched = sched_bytes(n_seqs) + bounds_bytes(total_tokens);
    if (fwd_bytes) *fwd_bytes = sched;
    if (bwd_bytes)
        *bwd_bytes = sched + align256(max_tiles(total_tokens, n_seqs) * n_heads * (size_t)(kTile * 16 * 2)) +
                     align256(sizeof(float) * max_tiles(total_tokens, n_seqs) * kTile * n_heads * padded_dim(head_dim));
    return DCP_OK;
}

// `merge` = false builds the work list over cu_seqlens itself and needs only sched_bytes of workspace
// (the entry point with built-in scratch, whose size cannot depend on the token count, uses it);
// the results are the same either way.
static int attn_fwd_impl(const char* fn, bool merge, const void* q, const void* k, const void* v,
                         const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen,
                         int32_t n_heads, int32_t head_dim, int64_t token_stride, int32_t causal, float softmax_scale,
                         void* o, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (int rc = check_shape(fn, n_seqs, total_tokens, max_seqlen, n_heads, head_dim, softmax_scale)) return rc;
    if (int rc = check_stride(fn, token_stride, n_heads, head_dim)) return rc;
    if (!cu_seqlens) return fail(DCP_ERR_INVALID_ARG, "%s: cu_seqlens is null", fn);
    if (!workspace) return fail(DCP_ERR_WORKSPACE, "%s: workspace is null", fn);
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return fail(DCP_ERR_WORKSPACE, "%s: workspace must be 256-byte aligned", fn);
    const size_t need = sched_bytes(n_seqs) + (merge ? bounds_bytes(total_tokens) : 0);
    if (workspace_bytes < need)
        return fail(DCP_ERR_WORKSPACE, "%s: workspace has %zu bytes, needs %zu", fn, workspace_bytes, need);
    if (total_tokens > 0 && (!q || !k || !v || !o || !lse)) return fail(DCP_ERR_INVALID_ARG, "%s: null tensor pointer", fn);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o))
        return fail(DCP_ERR_INVALID_ARG, "%s: tensor pointers must be 16-byte aligned", fn);
    DeviceInfo dev;
    if (int rc = device_info(&dev)) return rc;
    if (dev.cc_major != 10) return fail(DCP_ERR_UNSUPPORTED, "%s: this library runs on sm_100 devices only", fn);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    const SchedView sched = carve_sched(workspace, n_seqs);
    uint16_t* bounds = merge ? reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(workspace) + sched_bytes(n_seqs)) : nullptr;
    cudaError_t e;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)head_dim);
    if (short_sequence_path(n_seqs, total_tokens, max_seqlen)) {
        int32_t* first_seq = const_cast<int32_t*>(sched.order);      // the work list's arrays are free on this path
        {
            ScopedTimer t(DCP_KERNEL_PREP, stream);
            e = launch_small_check(false, cu_seqlens, n_seqs, total_tokens, max_seqlen, n_heads, sched.hdr, first_seq, dev.sm_count,
                                   stream);
        }
        if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: boundary check kernel: %s", fn, cudaGetErrorString(e));
        g_launches.fetch_add(1);
        if (total_tokens == 0 || n_seqs == 0) return DCP_OK;
        {
            ScopedTimer t(DCP_KERNEL_FWD, stream);
            e = launch_small_attn(false, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                  static_cast<const __nv_bfloat16*>(v), nullptr, lse, cu_seqlens, total_tokens, max_seqlen,
                                  n_heads, head_dim, token_stride, causal != 0, scale, static_cast<__nv_bfloat16*>(o), nullptr,
                                  nullptr, nullptr, sched.hdr, first_seq, dev.sm_count, stream);
        }
        if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: short-sequence kernel: %s", fn, cudaGetErrorString(e));
        g_launches.fetch_add(1);
        return DCP_OK;
    }
    const bool input_order = g_input_order.load() != 0;
    {
        ScopedTimer t(DCP_KERNEL_PREP, stream);
        e = launch_prep(cu_seqlens, n_seqs, total_tokens, max_seqlen, kFwdRowsPerItem, n_heads, sched, bounds, UINT32_MAX,
                        input_order, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: work-list kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(prep_launches(n_seqs, merge, input_order));
    if (total_tokens == 0 || n_seqs == 0) return DCP_OK;

    CUtensorMap tq, tk, tv, to;
    if (int rc = make_map(&tq, q, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tk, k, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tv, v, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&to, o, total_tokens, n_heads, head_dim, token_stride)) return rc;

    FwdParams p;
    p.cu_seqlens = merge ? sched.vcu : cu_seqlens;
    p.bounds = bounds;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.sched = sched;
    p.n_heads = n_heads;
    p.head_dim = head_dim;
    p.total_tokens = total_tokens;
    p.row_stride = token_stride;
    p.scale = scale;
    p.scale_log2 = p.scale * 1.4426950408889634f;
    {
        ScopedTimer t(DCP_KERNEL_FWD, stream);
        e = launch_attn_fwd(tq, tk, tv, to, p, head_dim, causal != 0, max_seqlen <= kShortItemMaxLen, dev.sm_count, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: attention kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(1);
    return DCP_OK;
}

extern "C" int dcp_varlen_attn_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                                   int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen, int32_t n_heads,
                                   int32_t head_dim, int32_t causal, float softmax_scale, void* o, float* lse,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return attn_fwd_impl("dcp_varlen_attn_fwd", true, q, k, v, cu_seqlens, n_seqs, total_tokens, max_seqlen, n_heads,
                         head_dim, (int64_t)n_heads * head_dim, causal, softmax_scale, o, lse, workspace, workspace_bytes,
                         cuda_stream);
}

extern "C" int dcp_varlen_attn_fwd_strided(const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                                           int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen, int32_t n_heads,
                                           int32_t head_dim, int64_t token_stride, int32_t causal, float softmax_scale,
                                           void* o, float* lse, void* workspace, size_t workspace_bytes,
                                           void* cuda_stream) {
    return attn_fwd_impl("dcp_varlen_attn_fwd_strided", true, q, k, v, cu_seqlens, n_seqs, total_tokens, max_seqlen,
                         n_heads, head_dim, token_stride, causal, softmax_scale, o, lse, workspace, workspace_bytes,
                         cuda_stream);
}

static int attn_bwd_impl(const char* fn, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                         const float* lse, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                         int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int64_t token_stride, int32_t causal,
                         float softmax_scale, void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes,
                         void* cuda_stream) {
    if (int rc = check_shape(fn, n_seqs, total_tokens, max_seqlen, n_heads, head_dim, softmax_scale)) return rc;
    if (int rc = check_stride(fn, token_stride, n_heads, head_dim)) return rc;
    if (!cu_seqlens) return fail(DCP_ERR_INVALID_ARG, "%s: cu_seqlens is null", fn);
    if (!workspace) return fail(DCP_ERR_WORKSPACE, "%s: workspace is null", fn);
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return fail(DCP_ERR_WORKSPACE, "%s: workspace must be 256-byte aligned", fn);
    size_t need = 0;
    dcp_varlen_attn_workspace(total_tokens, n_seqs, n_heads, head_dim, nullptr, &need);
    if (workspace_bytes < need) return fail(DCP_ERR_WORKSPACE, "%s: workspace has %zu bytes, needs %zu", fn, workspace_bytes, need);
    if (total_tokens > 0 && (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv))
        return fail(DCP_ERR_INVALID_ARG, "%s: null tensor pointer", fn);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return fail(DCP_ERR_INVALID_ARG, "%s: tensor pointers must be 16-byte aligned", fn);
    DeviceInfo dev;
    if (int rc = device_info(&dev)) return rc;
    if (dev.cc_major != 10) return fail(DCP_ERR_UNSUPPORTED, "%s: this library runs on sm_100 devices only", fn);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    const SchedView sched = carve_sched(workspace, n_seqs);
    uint16_t* bounds = reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(workspace) + sched_bytes(n_seqs));
    uint8_t* base = static_cast<uint8_t*>(workspace) + sched_bytes(n_seqs) + bounds_bytes(total_tokens);
    __nv_bfloat16* stats = reinterpret_cast<__nv_bfloat16*>(base);
    float* dq_acc = reinterpret_cast<float*>(base + align256(max_tiles(total_tokens, n_seqs) * n_heads * (size_t)(kTile * 16 * 2)));

    cudaError_t e;
    if (short_sequence_path(n_seqs, total_tokens, max_seqlen)) {
        int32_t* first_seq = const_cast<int32_t*>(sched.order);      // the work list's arrays are free on this path
        {
            ScopedTimer t(DCP_KERNEL_PREP, stream);
            e = launch_small_check(true, cu_seqlens, n_seqs, total_tokens, max_seqlen, n_heads, sched.hdr, first_seq, dev.sm_count,
                                   stream);
        }
        if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: boundary check kernel: %s", fn, cudaGetErrorString(e));
        g_launches.fetch_add(1);
        if (total_tokens == 0 || n_seqs == 0) return DCP_OK;
        {
            ScopedTimer t(DCP_KERNEL_BWD_MAIN, stream);
            e = launch_small_attn(true, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                  static_cast<const __nv_bfloat16*>(v), static_cast<const __nv_bfloat16*>(d_o),
                                  const_cast<float*>(lse), cu_seqlens, total_tokens, max_seqlen, n_heads, head_dim, token_stride,
                                  causal != 0, softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)head_dim), nullptr,
                                  static_cast<__nv_bfloat16*>(dq), static_cast<__nv_bfloat16*>(dk),
                                  static_cast<__nv_bfloat16*>(dv), sched.hdr, first_seq, dev.sm_count, stream);
        }
        if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: short-sequence kernel: %s", fn, cudaGetErrorString(e));
        g_launches.fetch_add(1);
        return DCP_OK;
    }
    const bool input_order = g_input_order.load() != 0;
    {
        ScopedTimer t(DCP_KERNEL_PREP, stream);
        e = launch_prep(cu_seqlens, n_seqs, total_tokens, max_seqlen, kTile, n_heads, sched, bounds,
                        (uint32_t)max_tiles(total_tokens, n_seqs), input_order, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: work-list kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(prep_launches(n_seqs, true, input_order));
    const int32_t* vcu = sched.vcu;      // every later kernel works on the virtual sequences
    if (total_tokens == 0 || n_seqs == 0) return DCP_OK;

    CUtensorMap tq, tk, tv, tg;
    if (int rc = make_map(&tq, q, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tk, k, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tv, v, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tg, d_o, total_tokens, n_heads, head_dim, token_stride)) return rc;
    CUtensorMap tdk, tdv;
    if (int rc = make_map(&tdk, dk, total_tokens, n_heads, head_dim, token_stride)) return rc;
    if (int rc = make_map(&tdv, dv, total_tokens, n_heads, head_dim, token_stride)) return rc;

    {
        ScopedTimer t(DCP_KERNEL_BWD_PRE, stream);
        e = launch_bwd_pre(static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse, vcu,
                           sched, stats, dq_acc, max_tiles(total_tokens, n_seqs) * kTile * n_heads * padded_dim(head_dim),
                           total_tokens, n_heads, head_dim, token_stride,
                           softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)head_dim), dev.sm_count, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: pre kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(1);

    BwdParams p;
    p.cu_seqlens = vcu;
    p.bounds = bounds;
    p.stats = stats;
    p.dq_acc = dq_acc;
    p.dq = static_cast<__nv_bfloat16*>(dq);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.sched = sched;
    p.n_heads = n_heads;
    p.head_dim = head_dim;
    p.total_tokens = total_tokens;
    p.row_stride = token_stride;
    p.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)head_dim);
    p.scale_log2 = p.scale * 1.4426950408889634f;
    {
        ScopedTimer t(DCP_KERNEL_BWD_MAIN, stream);
        e = launch_attn_bwd(tq, tk, tv, tg, tdk, tdv, p, head_dim, causal != 0, dev.sm_count, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: main kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(1);

    {
        ScopedTimer t(DCP_KERNEL_BWD_POST, stream);
        e = launch_bwd_post(dq_acc, static_cast<__nv_bfloat16*>(dq), vcu, sched, n_heads, head_dim, token_stride, p.scale,
                            dev.sm_count, stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: post kernel: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(1);
    return DCP_OK;
}

extern "C" int dcp_varlen_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                   const float* lse, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                                   int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int32_t causal,
                                   float softmax_scale, void* dq, void* dk, void* dv, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
    return attn_bwd_impl("dcp_varlen_attn_bwd", q, k, v, o, d_o, lse, cu_seqlens, n_seqs, total_tokens, max_seqlen, n_heads,
                         head_dim, (int64_t)n_heads * head_dim, causal, softmax_scale, dq, dk, dv, workspace, workspace_bytes,
                         cuda_stream);
}

extern "C" int dcp_varlen_attn_bwd_strided(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                           const float* lse, const int32_t* cu_seqlens, int32_t n_seqs,
                                           int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                                           int64_t token_stride, int32_t causal, float softmax_scale, void* dq, void* dk,
                                           void* dv, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return attn_bwd_impl("dcp_varlen_attn_bwd_strided", q, k, v, o, d_o, lse, cu_seqlens, n_seqs, total_tokens, max_seqlen,
                         n_heads, head_dim, token_stride, causal, softmax_scale, dq, dk, dv, workspace, workspace_bytes,
                         cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Forward attention for callers that cannot allocate device memory.
//
// The forward kernel needs scratch for its work list (header, CTA time spans, sequence order, prefix
// sums).  Here that scratch is a fixed array in the library's own device image, so the caller passes
// inputs and outputs only.  Every GPU that loads this library holds the array until the process exits.
#define DCP_NOALLOC_MAX_SEQS_VALUE 4096
namespace {
constexpr size_t kNoAllocScratchBytes = dcp::sched_bytes(DCP_NOALLOC_MAX_SEQS_VALUE);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code the array's name is only a handle, not a device address: ask the runtime for the
// address once per device, with that device current, and hand the kernels that pointer.  (The
// address is cached per device index for the life of the process; a cudaDeviceReset in between
// would make it stale.)
int noalloc_scratch(const char* fn, void** out) {
    static std::mutex mu;
    static void* scratch_of_device[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return fail(DCP_ERR_CUDA, "%s: cudaGetDevice failed or device index out of range", fn);
    std::lock_guard<std::mutex> lock(mu);
    if (!scratch_of_device[dev]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) return fail(DCP_ERR_CUDA, "%s: cudaGetSymbolAddress: %s", fn, cudaGetErrorString(e));
        scratch_of_device[dev] = ptr;
    }
    *out = scratch_of_device[dev];
    return DCP_OK;
}

// Reads the status word at `status_word`, reports it and clears it (the word is sticky on the device).
int report_status(void* status_word, cudaStream_t stream, const char* fn) {
    uint32_t status = 0;
    cudaError_t e = cudaMemcpyAsync(&status, status_word, sizeof status, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e == cudaSuccess && status != 0) {
        e = cudaMemsetAsync(status_word, 0, sizeof status, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    }
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: %s", fn, cudaGetErrorString(e));
    if (status == kStatusBadLengths)
        return fail(DCP_ERR_INVALID_ARG,
                    "cu_seqlens disagrees with n_seqs, total_tokens or max_seqlen (it must start at 0, never decrease, end "
                    "at total_tokens, and no sequence may exceed max_seqlen); that call computed nothing");
    if (status != 0) return fail(DCP_ERR_TIMEOUT, "a kernel abandoned a bounded wait (device status %u); results are invalid", status);
    return DCP_OK;
}
}  // namespace

extern "C" int dcp_varlen_attn_fwd_noalloc(const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                                           int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen, int32_t n_heads,
                                           int32_t head_dim, int32_t causal, float softmax_scale, void* o, float* lse,
                                           void* cuda_stream) {
    const char* fn = "dcp_varlen_attn_fwd_noalloc";
    if (n_seqs > DCP_NOALLOC_MAX_SEQS_VALUE)
        return fail(DCP_ERR_UNSUPPORTED, "%s: %d sequences exceed the built-in scratch (at most %d per call)", fn, n_seqs,
                    DCP_NOALLOC_MAX_SEQS_VALUE);
    if (n_seqs < 0) return fail(DCP_ERR_INVALID_ARG, "%s: negative n_seqs", fn);
    void* scratch = nullptr;
    if (int rc = noalloc_scratch(fn, &scratch)) return rc;
    if (sched_bytes(n_seqs) > kNoAllocScratchBytes)      // cannot happen for n_seqs <= the maximum; kept as a guard
        return fail(DCP_ERR_UNSUPPORTED, "%s: built-in scratch too small", fn);
    // short sequences are not merged here: the table that needs is sized by the token count
    return attn_fwd_impl(fn, false, q, k, v, cu_seqlens, n_seqs, total_tokens, max_seqlen, n_heads, head_dim,
                         (int64_t)n_heads * head_dim, causal, softmax_scale, o, lse, scratch, kNoAllocScratchBytes,
                         cuda_stream);
}

extern "C" int dcp_noalloc_status(void* cuda_stream) {
    void* scratch = nullptr;
    if (int rc = noalloc_scratch("dcp_noalloc_status", &scratch)) return rc;
    return report_status(scratch, static_cast<cudaStream_t>(cuda_stream), "dcp_noalloc_status");
}

extern "C" int dcp_query_status(void* workspace, void* cuda_stream) {
    if (!workspace) return fail(DCP_ERR_INVALID_ARG, "dcp_query_status: workspace is null");
    return report_status(workspace, static_cast<cudaStream_t>(cuda_stream), "dcp_query_status");
}

extern "C" int dcp_set_work_order(int input_order) {
    g_input_order.store(input_order ? 1 : 0);
    return DCP_OK;
}

extern "C" int dcp_set_short_sequence_path(int enabled) {
    g_short_path.store(enabled ? 1 : 0);
    return DCP_OK;
}

extern "C" int dcp_read_cta_spans(const void* workspace, int32_t which, void* cuda_stream, int64_t* begin_ns,
                                  int64_t* end_ns, int32_t* n_ctas) {
    if (!workspace || !begin_ns || !end_ns || !n_ctas || which < 0 || which > 1)
        return fail(DCP_ERR_INVALID_ARG, "dcp_read_cta_spans: null pointer or `which` not 0/1");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WorkspaceHeader hdr;
    static_assert(sizeof(CtaSpan) == 16, "span is two 64-bit words");
    std::vector<CtaSpan> spans(kMaxCtas);
    const uint8_t* base = static_cast<const uint8_t*>(workspace);
    cudaError_t e = cudaMemcpyAsync(&hdr, base, sizeof hdr, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(spans.data(), base + sizeof(WorkspaceHeader) + (size_t)which * kMaxCtas * sizeof(CtaSpan),
                            kMaxCtas * sizeof(CtaSpan), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "dcp_read_cta_spans: %s", cudaGetErrorString(e));
    if (hdr.magic[0] != kHeaderMagic0 || hdr.magic[1] != kHeaderMagic1 || hdr.n_ctas[which] > (uint32_t)kMaxCtas)
        return fail(DCP_ERR_INVALID_ARG, "dcp_read_cta_spans: no attention call has run on this workspace");
    *n_ctas = (int32_t)hdr.n_ctas[which];
    for (int i = 0; i < *n_ctas; ++i) {
        begin_ns[i] = (int64_t)spans[i].begin_ns;
        end_ns[i] = (int64_t)spans[i].end_ns;
    }
    return DCP_OK;
}

extern "C" int dcp_selftest_wait_timeout(void* workspace, uint32_t spin_limit, void* cuda_stream) {
    if (!workspace) return fail(DCP_ERR_WORKSPACE, "dcp_selftest_wait_timeout: workspace is null");
    if (spin_limit > (1u << 20)) return fail(DCP_ERR_INVALID_ARG, "dcp_selftest_wait_timeout: spin_limit above 2^20");
    const cudaError_t e = launch_wait_timeout_selftest(static_cast<WorkspaceHeader*>(workspace), spin_limit,
                                                       static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "dcp_selftest_wait_timeout: %s", cudaGetErrorString(e));
    g_launches.fetch_add(1);
    return DCP_OK;
}

extern "C" int dcp_copy_segments(const void* src, void* dst, const int32_t* seg, int32_t n_seg, int64_t row_bytes,
                                 int32_t n_planes, int64_t src_plane_bytes, int64_t dst_plane_bytes, int32_t reverse,
                                 void* cuda_stream) {
    const char* fn = "dcp_copy_segments";
    if (n_seg < 0 || n_planes < 1 || row_bytes < 4 || row_bytes % 4 != 0 || src_plane_bytes < 0 || dst_plane_bytes < 0 ||
        src_plane_bytes % 4 != 0 || dst_plane_bytes % 4 != 0)
        return fail(DCP_ERR_INVALID_ARG, "%s: sizes must be non-negative and multiples of 4 bytes", fn);
    if (n_planes > 65535) return fail(DCP_ERR_UNSUPPORTED, "%s: at most 65535 planes", fn);
    if (n_seg == 0) return DCP_OK;
    if (!src || !dst || !seg) return fail(DCP_ERR_INVALID_ARG, "%s: null pointer", fn);
    if ((reinterpret_cast<uintptr_t>(src) & 3u) || (reinterpret_cast<uintptr_t>(dst) & 3u))
        return fail(DCP_ERR_INVALID_ARG, "%s: tensors must be 4-byte aligned", fn);
    DeviceInfo dev;
    if (int rc = device_info(&dev)) return rc;
    const cudaError_t e = launch_copy_segments(src, dst, seg, n_seg, row_bytes, n_planes, src_plane_bytes, dst_plane_bytes,
                                               reverse != 0, dev.sm_count, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail(DCP_ERR_CUDA, "%s: %s", fn, cudaGetErrorString(e));
    g_launches.fetch_add(1);
    return DCP_OK;
}

extern "C" int dcp_profile_enable(int on) {
    g_prof_on.store(on ? 1 : 0);
    return DCP_OK;
}

extern "C" int dcp_profile_read(float* ms, int64_t* launches) {
    if (!ms || !launches) return fail(DCP_ERR_INVALID_ARG, "dcp_profile_read: null pointer");
    std::vector<TimedLaunch> pending;
    {
        std::lock_guard<std::mutex> lock(g_prof_mu);
        pending.swap(g_prof_pending);
    }
    for (int i = 0; i < DCP_N_KERNELS; ++i) { ms[i] = 0.f; launches[i] = 0; }
    int rc = DCP_OK;
    for (const TimedLaunch& t : pending) {
        float one = 0.f;
        cudaError_t e = cudaEventSynchronize(t.stop);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&one, t.start, t.stop);
        if (e != cudaSuccess) rc = fail(DCP_ERR_CUDA, "dcp_profile_read: %s", cudaGetErrorString(e));
        else { ms[t.kernel] += one; launches[t.kernel] += 1; }
    }
    std::lock_guard<std::mutex> lock(g_prof_mu);
    for (const TimedLaunch& t : pending) {
        g_event_pool[t.device].push_back(t.start);
        g_event_pool[t.device].push_back(t.stop);
    }
    return rc;
}
