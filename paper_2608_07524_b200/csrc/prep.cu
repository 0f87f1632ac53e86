// Work-list construction and the two small memory-bound backward helpers.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sched.cuh"

namespace dcp {

constexpr int kPrepThreads = 1024;

// One CTA.  order[] = sequence ids sorted by (length descending, id ascending) via a rank sort;
// prefix[i] = number of work items of the first i sequences in that order, where a sequence of
// length L contributes ceil(L / rows_per_block) * n_heads items.
__global__ void __launch_bounds__(kPrepThreads) prep_kernel(const int32_t* __restrict__ cu, int32_t n_seqs,
                                                            int32_t rows_per_block, int32_t n_heads,
                                                            WorkspaceHeader* hdr, int32_t* order, uint32_t* prefix,
                                                            uint32_t* tile_prefix) {
    __shared__ uint32_t chunk_sum[kPrepThreads];
    const int tid = threadIdx.x;
    for (int i = tid; i < n_seqs; i += kPrepThreads) {
        const int32_t len_i = cu[i + 1] - cu[i];
        int rank = 0;
        for (int j = 0; j < n_seqs; ++j) {
            const int32_t len_j = cu[j + 1] - cu[j];
            rank += (len_j > len_i) || (len_j == len_i && j < i);
        }
        order[rank] = i;
    }
    __syncthreads();
    // exclusive scan of item counts over the sorted order: contiguous chunk per thread
    const int per = (n_seqs + kPrepThreads - 1) / kPrepThreads;
    const int begin = tid * per, end = min(begin + per, n_seqs);
    auto items_of = [&](int pos) -> uint32_t {
        const int s = order[pos];
        const int32_t len = cu[s + 1] - cu[s];
        return (uint32_t)((len + rows_per_block - 1) / rows_per_block) * (uint32_t)n_heads;
    };
    uint32_t local = 0;
    for (int i = begin; i < end; ++i) local += items_of(i);
    chunk_sum[tid] = local;
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0;
        for (int i = 0; i < kPrepThreads; ++i) {
            const uint32_t c = chunk_sum[i];
            chunk_sum[i] = run;
            run += c;
        }
        prefix[n_seqs] = run;
        hdr->n_items = run;
        hdr->work_counter = 0;
        hdr->status = 0;
    }
    __syncthreads();
    uint32_t run = chunk_sum[tid];
    for (int i = begin; i < end; ++i) {
        prefix[i] = run;
        run += items_of(i);
    }
    __syncthreads();
    // tile_prefix[b] = number of 128-row tiles of sequences 0..b-1 (input order): same two-level scan
    auto tiles_of = [&](int b) -> uint32_t { return (uint32_t)((cu[b + 1] - cu[b] + kTile - 1) / kTile); };
    local = 0;
    for (int i = begin; i < end; ++i) local += tiles_of(i);
    chunk_sum[tid] = local;
    __syncthreads();
    if (tid == 0) {
        uint32_t acc = 0;
        for (int i = 0; i < kPrepThreads; ++i) {
            const uint32_t c = chunk_sum[i];
            chunk_sum[i] = acc;
            acc += c;
        }
        tile_prefix[n_seqs] = acc;
    }
    __syncthreads();
    run = chunk_sum[tid];
    for (int i = begin; i < end; ++i) {
        tile_prefix[i] = run;
        run += tiles_of(i);
    }
}

cudaError_t launch_prep(const int32_t* cu_seqlens, int32_t n_seqs, int32_t rows_per_block, int32_t n_heads,
                        const SchedView& sched, cudaStream_t stream) {
    prep_kernel<<<1, kPrepThreads, 0, stream>>>(cu_seqlens, n_seqs, rows_per_block, n_heads, sched.hdr,
                                                const_cast<int32_t*>(sched.order), const_cast<uint32_t*>(sched.prefix),
                                                const_cast<uint32_t*>(sched.tile_prefix));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Backward helper 1.  For every (128-row tile, head) it writes a [128 rows x 16] bf16 tile holding,
// per query row, -lse/scale (columns 0-2) and -D_i = -sum_c dO_ic O_ic (columns 8-10), each split
// into three bf16 parts whose sum carries 24 bits; the main kernel adds them to its score and dP
// accumulators with a K=16 MMA against a tile of ones.  Rows past the sequence end get -1e30 and 0,
// which makes their probabilities vanish without masking.  The tile is stored in the MMA's shared-
// memory layout (8x8 core matrices; column halves 2048 bytes apart) and is 4 KB-aligned, so one bulk
// copy fetches it.  Also zeroes the fp32 dQ accumulator.  HBM-bound.
template <int D>
__global__ void __launch_bounds__(256) bwd_pre_kernel(const __nv_bfloat16* __restrict__ o,
                                                      const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ lse,
                                                      const int32_t* __restrict__ cu, const uint32_t* __restrict__ tile_prefix,
                                                      int32_t n_seqs, __nv_bfloat16* __restrict__ stats,
                                                      float* __restrict__ dq_acc, size_t dq_acc_vec4,
                                                      int32_t total_tokens, int32_t n_heads, float inv_scale) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_blocks = tile_prefix[n_seqs] * (uint32_t)n_heads;
    for (uint32_t blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
        const uint32_t t = blk / n_heads, h = blk % n_heads;
        int lo = 0, hi = n_seqs;                              // sequence owning tile t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (tile_prefix[mid] <= t) lo = mid; else hi = mid;
        }
        while (lo + 1 < n_seqs && tile_prefix[lo + 1] <= t) ++lo;   // skip empty sequences
        const int row0 = (int)(t - tile_prefix[lo]) * kTile;
        const int len = cu[lo + 1] - cu[lo];
        uint8_t* out = reinterpret_cast<uint8_t*>(stats) + (size_t)blk * (kTile * 16 * 2);
        for (int r = warp; r < kTile; r += 8) {
            float acc = 0.f, nl = -1e30f;
            if (row0 + r < len) {
                const size_t tok = (size_t)cu[lo] + row0 + r;
                const size_t row = tok * n_heads + h;
                constexpr int kPer = D / 32;           // elements per lane: 2 or 4
                const __nv_bfloat16* po = o + row * D + lane * kPer;
                const __nv_bfloat16* pg = d_o + row * D + lane * kPer;
                if (kPer == 4) {
                    const uint2 a = *reinterpret_cast<const uint2*>(po), b = *reinterpret_cast<const uint2*>(pg);
                    const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.x));
                    const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.y));
                    const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.x));
                    const float2 b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.y));
                    acc = a0.x * b0.x + a0.y * b0.y + a1.x * b1.x + a1.y * b1.y;
                } else {
                    const uint32_t a = *reinterpret_cast<const uint32_t*>(po), b = *reinterpret_cast<const uint32_t*>(pg);
                    const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a));
                    const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b));
                    acc = a0.x * b0.x + a0.y * b0.y;
                }
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
                nl = -lse[(size_t)h * total_tokens + tok] * inv_scale;
            }
            if (lane < 2) {     // lane 0: the lse term into column half 0; lane 1: the D term into half 1
                const float x = lane == 0 ? nl : -acc;
                const __nv_bfloat16 b0 = __float2bfloat16(x);
                const float r1 = x - __bfloat162float(b0);
                const __nv_bfloat16 b1 = __float2bfloat16(r1);
                const __nv_bfloat16 b2 = __float2bfloat16(r1 - __bfloat162float(b1));
                uint4 v;
                v.x = (uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
                v.y = (uint32_t)__bfloat16_as_ushort(b2);
                v.z = 0u;
                v.w = 0u;
                *reinterpret_cast<uint4*>(out + lane * 2048 + (r / 8) * 128 + (r % 8) * 16) = v;
            }
        }
    }
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < dq_acc_vec4; i += stride)
        reinterpret_cast<float4*>(dq_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

cudaError_t launch_bwd_pre(const __nv_bfloat16* o, const __nv_bfloat16* d_o, const float* lse, const int32_t* cu_seqlens,
                           const SchedView& sched, __nv_bfloat16* stats, float* dq_acc, size_t dq_acc_elems,
                           int32_t total_tokens, int32_t n_heads, int32_t head_dim, float scale, int n_sms,
                           cudaStream_t stream) {
    const int blocks = n_sms * 8;
    if (head_dim == 128)
        bwd_pre_kernel<128><<<blocks, 256, 0, stream>>>(o, d_o, lse, cu_seqlens, sched.tile_prefix, sched.n_seqs, stats,
                                                        dq_acc, dq_acc_elems / 4, total_tokens, n_heads, 1.0f / scale);
    else
        bwd_pre_kernel<64><<<blocks, 256, 0, stream>>>(o, d_o, lse, cu_seqlens, sched.tile_prefix, sched.n_seqs, stats,
                                                       dq_acc, dq_acc_elems / 4, total_tokens, n_heads, 1.0f / scale);
    return cudaGetLastError();
}

// Backward helper 2: dq[T, H, d] = bf16(scale * dq_acc).  dq_acc holds, per (tile, head), a block
// [d/4][128 rows][4 floats]; a CTA reads one block with coalesced 16-byte loads, transposes it in
// shared memory as bf16 and writes whole rows.  Rows past the sequence end are skipped.
template <int D>
__global__ void __launch_bounds__(256) bwd_post_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq,
                                                       const int32_t* __restrict__ cu, const uint32_t* __restrict__ tile_prefix,
                                                       int32_t n_seqs, int32_t n_heads, float scale) {
    constexpr int kRowBytes = D * 2 + 16;                    // padded row of bf16
    __shared__ __align__(16) uint8_t tile[kTile * kRowBytes];
    const uint32_t n_tiles = tile_prefix[n_seqs];
    const uint32_t n_blocks = n_tiles * (uint32_t)n_heads;
    for (uint32_t blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
        const uint32_t t = blk / n_heads, h = blk % n_heads;
        int lo = 0, hi = n_seqs;                              // sequence owning tile t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (tile_prefix[mid] <= t) lo = mid; else hi = mid;
        }
        while (lo + 1 < n_seqs && tile_prefix[lo + 1] <= t) ++lo;   // skip empty sequences
        const int row0 = (int)(t - tile_prefix[lo]) * kTile;
        const int len = cu[lo + 1] - cu[lo];
        const int rows = min(kTile, len - row0);
        const float4* src = reinterpret_cast<const float4*>(dq_acc + (size_t)blk * (kTile * D));
        for (int e = threadIdx.x; e < kTile * D / 4; e += blockDim.x) {
            const int c4 = e / kTile, r = e % kTile;
            const float4 v = src[e];
            __nv_bfloat162 lo2 = __floats2bfloat162_rn(v.x * scale, v.y * scale);
            __nv_bfloat162 hi2 = __floats2bfloat162_rn(v.z * scale, v.w * scale);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo2);
            pk.y = *reinterpret_cast<uint32_t*>(&hi2);
            *reinterpret_cast<uint2*>(tile + r * kRowBytes + c4 * 8) = pk;
        }
        __syncthreads();
        constexpr int kChunks = D * 2 / 16;                  // 16-byte chunks per row
        for (int e = threadIdx.x; e < rows * kChunks; e += blockDim.x) {
            const int r = e / kChunks, c = e % kChunks;
            const uint4 v = *reinterpret_cast<const uint4*>(tile + r * kRowBytes + c * 16);
            __nv_bfloat16* out = dq + (((size_t)cu[lo] + row0 + r) * n_heads + h) * D;
            reinterpret_cast<uint4*>(out)[c] = v;
        }
        __syncthreads();
    }
}

cudaError_t launch_bwd_post(const float* dq_acc, __nv_bfloat16* dq, const int32_t* cu_seqlens, const SchedView& sched,
                            int32_t n_heads, int32_t head_dim, float scale, int n_sms, cudaStream_t stream) {
    const int blocks = n_sms * 4;
    if (head_dim == 128)
        bwd_post_kernel<128><<<blocks, 256, 0, stream>>>(dq_acc, dq, cu_seqlens, sched.tile_prefix, sched.n_seqs, n_heads, scale);
    else
        bwd_post_kernel<64><<<blocks, 256, 0, stream>>>(dq_acc, dq, cu_seqlens, sched.tile_prefix, sched.n_seqs, n_heads, scale);
    return cudaGetLastError();
}

}  // namespace dcp
