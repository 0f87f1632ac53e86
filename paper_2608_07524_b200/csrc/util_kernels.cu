// Small helper kernels: row-range copies that move a micro-batch's sequences between a batch and the
// micro-batch's own packed tensors, and the self-test of the bounded-wait abort path.
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sched.cuh"
#include "sm100_ptx.cuh"

namespace dcp {

// seg holds n_seg triples (a, b, rows).  Forward: rows [b, b + rows) of dst = rows [a, a + rows) of src;
// reverse: rows [a, a + rows) of dst = rows [b, b + rows) of src, so that the triples that gathered a
// micro-batch also scatter its results back.  A row is row_bytes bytes; blockIdx.y selects a plane.
// One CTA per (segment, plane), grid-stride over segments; the caller keeps segments short enough
// (a few hundred KB) for the grid to balance.  VEC = uint4 when everything is 16-byte aligned.
template <typename VEC>
__global__ void __launch_bounds__(256) copy_segments_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst,
                                                            const int32_t* __restrict__ seg, int32_t n_seg,
                                                            int64_t row_bytes, int64_t src_plane_bytes,
                                                            int64_t dst_plane_bytes, int reverse) {
    const uint8_t* s_plane = src + (size_t)blockIdx.y * (size_t)src_plane_bytes;
    uint8_t* d_plane = dst + (size_t)blockIdx.y * (size_t)dst_plane_bytes;
    for (int32_t i = blockIdx.x; i < n_seg; i += gridDim.x) {
        const int32_t a = seg[3 * i], b = seg[3 * i + 1], rows = seg[3 * i + 2];
        if (rows <= 0 || a < 0 || b < 0) continue;
        const VEC* s = reinterpret_cast<const VEC*>(s_plane + (size_t)(reverse ? b : a) * (size_t)row_bytes);
        VEC* d = reinterpret_cast<VEC*>(d_plane + (size_t)(reverse ? a : b) * (size_t)row_bytes);
        const size_t n = (size_t)rows * (size_t)row_bytes / sizeof(VEC);
        size_t e = threadIdx.x;
        for (; e + 3 * 256 < n; e += 4 * 256) {          // four independent loads in flight per thread
            const VEC v0 = s[e], v1 = s[e + 256], v2 = s[e + 512], v3 = s[e + 768];
            d[e] = v0; d[e + 256] = v1; d[e + 512] = v2; d[e + 768] = v3;
        }
        for (; e < n; e += 256) d[e] = s[e];
    }
}

cudaError_t launch_copy_segments(const void* src, void* dst, const int32_t* seg, int32_t n_seg, int64_t row_bytes,
                                 int32_t n_planes, int64_t src_plane_bytes, int64_t dst_plane_bytes, bool reverse,
                                 int n_sms, cudaStream_t stream) {
    const bool wide = row_bytes % 16 == 0 && src_plane_bytes % 16 == 0 && dst_plane_bytes % 16 == 0 &&
                      (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0;
    int bx = n_sms * 8 / n_planes;
    if (bx < 1) bx = 1;
    if (bx > n_seg) bx = n_seg;
    const dim3 grid((unsigned)bx, (unsigned)n_planes);
    if (wide)
        copy_segments_kernel<uint4><<<grid, 256, 0, stream>>>(static_cast<const uint8_t*>(src), static_cast<uint8_t*>(dst), seg,
                                                              n_seg, row_bytes, src_plane_bytes, dst_plane_bytes, reverse);
    else
        copy_segments_kernel<uint32_t><<<grid, 256, 0, stream>>>(static_cast<const uint8_t*>(src), static_cast<uint8_t*>(dst),
                                                                 seg, n_seg, row_bytes, src_plane_bytes, dst_plane_bytes, reverse);
    return cudaGetLastError();
}

// One warp waits on a barrier that nothing ever arrives at, with the attention kernels' own wait helper
// and a caller-chosen poll limit, then leaves normally: the wait gives up, raises the abort flag and the
// status word, and the kernel returns.
__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(WorkspaceHeader* hdr, uint32_t spin_limit) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_mbar_init();
        header_begin_call(hdr, false);
    }
    __syncwarp();
    const WaitGuard guard{&abort_flag, &hdr->status};
    if (threadIdx.x == 0) mbar_wait_limited(&bar, 0, guard, spin_limit);      // phase 0 never completes
    __syncwarp();
    // every later wait of the CTA returns at once, which is what lets a real kernel run to its end
    mbar_wait_limited(&bar, 0, guard, 1u << 20);
}

cudaError_t launch_wait_timeout_selftest(WorkspaceHeader* hdr, uint32_t spin_limit, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(hdr, spin_limit);
    return cudaGetLastError();
}

}  // namespace dcp
