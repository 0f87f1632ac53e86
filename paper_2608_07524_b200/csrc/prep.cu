// Work-list construction and the two small memory-bound backward helpers.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sched.cuh"

namespace dcp {

constexpr int kPrepThreads = 1024;
constexpr int kRankInKernelMax = 256;     // above this many sequences the rank sort runs over several CTAs (rank_kernel)

__device__ inline uint32_t block_exclusive_scan(uint32_t v, uint32_t* scratch, uint32_t* total);
__device__ inline int block_exclusive_max_scan(int v, int* scratch);

// Merging of short sequences into virtual sequences of at most 128 tokens.  One CTA.
//
// A sequence is "short" if length <= max_short (empty ones included).  Two local rules say when a short
// sequence joins the virtual sequence of its short predecessor:
//   rule 0: both START in the same window of `window` = 129 - max_short packed positions, so a virtual
//           sequence spans at most (window - 1) + max_short = 128 tokens;
//   rule 1: the predecessor's first and this sequence's last token lie in the same ALIGNED window of 128
//           positions, so a virtual sequence lies inside one such window (sequences that cross a window
//           boundary stay alone).
// Rule 0 fills tiles well when sequences are much shorter than 64 tokens, rule 1 when they are close to
// 64 and aligned (64-token sequences pair up exactly, which their start windows of 65 almost never allow).
// Both are local (whether a sequence starts a virtual sequence depends on it and its predecessor only),
// so heads are found in parallel and compacted with a scan; the kernel counts the heads under both rules
// and keeps the rule that gives fewer (rule 1 only if the batch has no empty sequence, which keeps the
// bound on the number of tiles that sizes the workspace: it is derived for rule 0).
// Outputs: vcu[0..n_v] = boundaries of the virtual sequences, vcu[n_v+1..n_seqs] = total_tokens
// (empty padding, so that vcu is a valid boundary array of n_seqs sequences); hdr->n_vseq = n_v;
// hdr->merge_rule = the rule used; vstart[i] = first token of the virtual sequence that input
// sequence i belongs to (read by bounds_kernel, so that no thread there has to walk back over a run,
// which under rule 0 may hold any number of empty sequences).
__device__ __forceinline__ bool merge_is_head(const int32_t* __restrict__ cu, int i, int32_t max_short, uint32_t rule) {
    if (i == 0 || cu[i + 1] - cu[i] > max_short || cu[i] - cu[i - 1] > max_short) return true;
    if (rule == 0) {
        const int window = kTile + 1 - max_short;
        return cu[i - 1] / window != cu[i] / window;
    }
    return cu[i - 1] / kTile != (cu[i + 1] - 1) / kTile;
}

__global__ void __launch_bounds__(kPrepThreads) merge_kernel(const int32_t* __restrict__ cu, int32_t n_seqs,
                                                             int32_t total_tokens, int32_t max_short,
                                                             WorkspaceHeader* hdr, int32_t* vcu, int32_t* vstart) {
    __shared__ uint32_t scratch[33];
    const int tid = threadIdx.x;
    const int per = (n_seqs + kPrepThreads - 1) / kPrepThreads;
    const int begin = min(tid * per, n_seqs), end = min(begin + per, n_seqs);
    // The boundaries come from the caller and index everything that follows: they must start at 0, never
    // decrease and end at total_tokens.  If not, the status word says so and every sequence is made empty,
    // which turns the rest of the call into no-ops.  This kernel is the first of a call.
    int bad = (tid == 0 && (cu[0] != 0 || cu[n_seqs] != total_tokens)) ? 1 : 0;
    for (int i = begin; i < end; ++i) bad |= cu[i + 1] < cu[i] ? 1 : 0;
    bad = __syncthreads_or(bad);
    if (tid == 0) header_begin_call(hdr, bad != 0);
    if (bad) {
        for (int i = tid; i <= n_seqs; i += kPrepThreads) vcu[i] = 0;
        if (tid == 0) hdr->n_vseq = 0;
        return;
    }
    uint32_t local0 = 0, local1 = 0, n_v0 = 0, n_v1 = 0;
    int empty = 0;
    for (int i = begin; i < end; ++i) {
        local0 += merge_is_head(cu, i, max_short, 0) ? 1u : 0u;
        local1 += merge_is_head(cu, i, max_short, 1) ? 1u : 0u;
        empty |= cu[i + 1] == cu[i] ? 1 : 0;
    }
    empty = __syncthreads_or(empty);
    const uint32_t run0 = block_exclusive_scan(local0, scratch, &n_v0);
    const uint32_t run1 = block_exclusive_scan(local1, scratch, &n_v1);
    const uint32_t rule = (!empty && n_v1 < n_v0) ? 1u : 0u;
    const uint32_t n_v = rule ? n_v1 : n_v0;
    uint32_t run = rule ? run1 : run0;
    if (tid == 0) {
        hdr->n_vseq = n_v;
        hdr->merge_rule = rule;
    }
    int last_head = -1;
    for (int i = begin; i < end; ++i)
        if (merge_is_head(cu, i, max_short, rule)) {
            vcu[run++] = cu[i];
            last_head = i;
        }
    for (uint32_t i = n_v + tid; i <= (uint32_t)n_seqs; i += kPrepThreads) vcu[i] = total_tokens;
    // head of the run each sequence belongs to: the last head at or before it (sequence 0 is always one)
    int cur = block_exclusive_max_scan(last_head, reinterpret_cast<int*>(scratch));
    for (int i = begin; i < end; ++i) {
        if (merge_is_head(cu, i, max_short, rule)) cur = i;
        vstart[i] = cu[cur];
    }
}

// One warp per input sequence of at most 128 tokens, over as many CTAs as needed: bounds[t] for
// each of its tokens t = (first, end) position of the sequence relative to the start of its virtual
// sequence, one byte each (the lanes write consecutive tokens).  merge_kernel has left that start in vstart[].
__global__ void __launch_bounds__(256) bounds_kernel(const int32_t* __restrict__ cu, int32_t n_seqs,
                                                     const WorkspaceHeader* __restrict__ hdr,
                                                     const int32_t* __restrict__ vstart, uint16_t* __restrict__ bounds) {
    const int i = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (i >= n_seqs || hdr->call_bad) return;      // merge_kernel found the boundaries inconsistent
    const int32_t a = cu[i], b = cu[i + 1];
    if (b == a || b - a > kTile) return;
    const int32_t v0 = vstart[i];
    const uint16_t packed = (uint16_t)((a - v0) | ((b - v0) << 8));
    for (int32_t t = a + lane; t < b; t += 32) bounds[t] = packed;
}

// Rank sort, one thread per sequence over as many CTAs as needed: order[] = sequence ids sorted by
// (length descending, id ascending).  Used on its own for batches of more than kRankInKernelMax
// sequences (one CTA doing it for a thousand sequences takes 37 us, eight CTAs 4 us); small batches do the
// same loop inside prep_kernel and save the launch.  Sequences
// from *n_live on (if given) are empty padding: they keep their own index as rank and are not
// compared against.
__global__ void __launch_bounds__(256) rank_kernel(const int32_t* __restrict__ cu, int32_t n_seqs,
                                                   const uint32_t* __restrict__ n_live_ptr, int32_t* order) {
    __shared__ int32_t len_tile[256];
    const int n_live = n_live_ptr ? min((int)*n_live_ptr, n_seqs) : n_seqs;
    const int i = blockIdx.x * 256 + threadIdx.x;
    if ((int)blockIdx.x * 256 >= n_live) {             // a whole block of padding
        if (i < n_seqs) order[i] = i;
        return;
    }
    const int32_t len_i = i < n_seqs ? cu[i + 1] - cu[i] : 0;
    int rank = i > n_live ? i - n_live : 0;             // padding before i, all of length 0 like i itself
    for (int j0 = 0; j0 < n_live; j0 += 256) {
        const int j = j0 + threadIdx.x;
        __syncthreads();
        len_tile[threadIdx.x] = j < n_live ? cu[j + 1] - cu[j] : -1;     // -1 never outranks anything
        __syncthreads();
        const int cnt = min(256, n_live - j0);
        for (int t = 0; t < cnt; ++t) {
            const int32_t len_j = len_tile[t];
            rank += (len_j > len_i) || (len_j == len_i && j0 + t < i);
        }
    }
    if (i < n_seqs) order[rank] = i;
}

// Exclusive prefix sum of one value per thread over a CTA of kPrepThreads threads; *total receives
// the sum.  scratch holds 33 words.
__device__ inline uint32_t block_exclusive_scan(uint32_t v, uint32_t* scratch, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += t;
    }
    __syncthreads();                       // scratch may still be read from an earlier call
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const uint32_t w = scratch[lane];
        uint32_t wi = w;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, wi, s);
            if (lane >= s) wi += t;
        }
        scratch[lane] = wi - w;
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    *total = scratch[32];
    return scratch[warp] + incl - v;
}

// Exclusive running maximum of one value per thread (in thread order) over a CTA of kPrepThreads
// threads; -1 where nothing precedes.  scratch holds 33 words.
__device__ inline int block_exclusive_max_scan(int v, int* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl = max(incl, t);
    }
    __syncthreads();                       // scratch may still be read from an earlier scan
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int wi = scratch[lane];
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, s);
            if (lane >= s) wi = max(wi, t);
        }
        scratch[lane] = wi;                // inclusive over warps
    }
    __syncthreads();
    int excl = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) excl = -1;
    if (warp > 0) excl = max(excl, scratch[warp - 1]);
    return excl;
}

// One CTA.  order[] as above (computed here if `ranked` is 0, by rank_kernel if 1; 2 keeps the input
// order, a measurement aid); prefix[i] = number of work items of the
// first i sequences in that order, where a sequence of length L contributes
// ceil(L / rows_per_block) * n_heads items; tile_prefix[b] = 128-row tiles before sequence b.
// Sequences from *n_live_ptr on (if given) are empty padding and sorted last: only the live ones
// are scanned, the rest get the totals.
__global__ void __launch_bounds__(kPrepThreads) prep_kernel(const int32_t* __restrict__ cu, int32_t n_seqs,
                                                            const uint32_t* __restrict__ n_live_ptr,
                                                            int32_t rows_per_block, int32_t n_heads,
                                                            WorkspaceHeader* hdr, int32_t* order, uint32_t* prefix,
                                                            uint32_t* tile_prefix, int ranked, int32_t total_tokens,
                                                            uint32_t tile_capacity) {
    __shared__ uint32_t scratch[33];
    __shared__ int32_t len_sh[kPrepThreads];
    const int tid = threadIdx.x;
    const int n_live = n_live_ptr ? min((int)*n_live_ptr, n_seqs) : n_seqs;
    if (!n_live_ptr) {
        // no merge_kernel ran before: check the caller's boundaries here (see merge_kernel)
        int bad = (tid == 0 && (cu[0] != 0 || cu[n_seqs] != total_tokens)) ? 1 : 0;
        for (int i = tid; i < n_seqs; i += kPrepThreads) bad |= cu[i + 1] < cu[i] ? 1 : 0;
        bad = __syncthreads_or(bad);
        if (tid == 0) header_begin_call(hdr, bad != 0);
        if (bad) {
            for (int i = tid; i <= n_seqs; i += kPrepThreads) { prefix[i] = 0; tile_prefix[i] = 0; }
            for (int i = tid; i < n_seqs; i += kPrepThreads) order[i] = i;
            if (tid == 0) { hdr->n_items = 0; hdr->work_counter = 0; }
            return;
        }
    }
    if (ranked == 2) {
        for (int i = tid; i < n_seqs; i += kPrepThreads) order[i] = i;
    } else if (!ranked) {                             // n_seqs <= kRankInKernelMax: one sequence per thread
        len_sh[tid] = tid < n_seqs ? cu[tid + 1] - cu[tid] : -1;
        __syncthreads();
        if (tid < n_seqs) {
            const int32_t len_i = len_sh[tid];
            int rank = 0;
            for (int j = 0; j < n_seqs; ++j) {
                const int32_t len_j = len_sh[j];
                rank += (len_j > len_i) || (len_j == len_i && j < tid);
            }
            order[rank] = tid;
        }
    }
    __syncthreads();
    // exclusive scan of item counts over the sorted order: contiguous chunk per thread
    const int per = (n_live + kPrepThreads - 1) / kPrepThreads;
    const int begin = min(tid * per, n_live), end = min(begin + per, n_live);
    auto items_of = [&](int pos) -> uint32_t {
        const int s = order[pos];
        const int32_t len = cu[s + 1] - cu[s];
        return (uint32_t)((len + rows_per_block - 1) / rows_per_block) * (uint32_t)n_heads;
    };
    uint32_t local = 0, total = 0;
    for (int i = begin; i < end; ++i) local += items_of(i);
    uint32_t run = block_exclusive_scan(local, scratch, &total);
    for (int i = begin; i < end; ++i) {
        prefix[i] = run;
        run += items_of(i);
    }
    for (int i = n_live + tid; i <= n_seqs; i += kPrepThreads) prefix[i] = total;
    if (tid == 0) {
        hdr->n_items = total;
        hdr->work_counter = 0;
    }
    // tile_prefix[b] = number of 128-row tiles of sequences 0..b-1 (input order): same two-level scan
    auto tiles_of = [&](int b) -> uint32_t { return (uint32_t)((cu[b + 1] - cu[b] + kTile - 1) / kTile); };
    local = 0;
    for (int i = begin; i < end; ++i) local += tiles_of(i);
    run = block_exclusive_scan(local, scratch, &total);
    if (total > tile_capacity) {
        // more tiles than the workspace was sized for: max_seqlen was understated (the bound on merged runs
        // relies on it).  Nothing may index the per-tile storage: no items, no tiles.
        for (int i = tid; i <= n_seqs; i += kPrepThreads) tile_prefix[i] = 0;
        if (tid == 0) {
            hdr->n_items = 0;
            atomicMax(&hdr->status, (uint32_t)kStatusBadLengths);
        }
        return;
    }
    for (int i = begin; i < end; ++i) {
        tile_prefix[i] = run;
        run += tiles_of(i);
    }
    for (int i = n_live + tid; i <= n_seqs; i += kPrepThreads) tile_prefix[i] = total;
}

int prep_launches(int32_t n_seqs, bool merge, bool input_order) {
    return (n_seqs > kRankInKernelMax && !input_order ? 2 : 1) + (merge ? (n_seqs > 0 ? 2 : 1) : 0);
}

cudaError_t launch_prep(const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen,
                        int32_t rows_per_block, int32_t n_heads, const SchedView& sched, uint16_t* bounds,
                        uint32_t tile_capacity, bool input_order, cudaStream_t stream) {
    const int32_t* cu = cu_seqlens;
    const uint32_t* n_live = nullptr;
    if (bounds) {                                       // merge short sequences; everything below sees vcu
        const int32_t max_short = max_seqlen < kMergeMaxLen ? (max_seqlen > 0 ? max_seqlen : 1) : kMergeMaxLen;
        // order[] is not needed until the ranking below: until then it carries each sequence's run start
        merge_kernel<<<1, kPrepThreads, 0, stream>>>(cu_seqlens, n_seqs, total_tokens, max_short, sched.hdr,
                                                     const_cast<int32_t*>(sched.vcu), const_cast<int32_t*>(sched.order));
        if (cudaError_t e = cudaGetLastError()) return e;
        if (n_seqs > 0)
            bounds_kernel<<<(n_seqs + 7) / 8, 256, 0, stream>>>(cu_seqlens, n_seqs, sched.hdr, sched.order, bounds);
        if (cudaError_t e = cudaGetLastError()) return e;
        cu = sched.vcu;
        n_live = &sched.hdr->n_vseq;
    }
    const int ranked = input_order ? 2 : (n_seqs > kRankInKernelMax ? 1 : 0);
    if (ranked == 1) {
        rank_kernel<<<(n_seqs + 255) / 256, 256, 0, stream>>>(cu, n_seqs, n_live, const_cast<int32_t*>(sched.order));
        if (cudaError_t e = cudaGetLastError()) return e;
    }
    prep_kernel<<<1, kPrepThreads, 0, stream>>>(cu, n_seqs, n_live, rows_per_block, n_heads, sched.hdr,
                                                const_cast<int32_t*>(sched.order), const_cast<uint32_t*>(sched.prefix),
                                                const_cast<uint32_t*>(sched.tile_prefix), ranked, total_tokens, tile_capacity);
    return cudaGetLastError();
}

// The sequence that owns 128-row tile t: (sequence, first row of the tile inside it, its length, its first token).
// A binary search of dependent loads, a few microseconds when they miss L1: the helper kernels below look up the
// NEXT block's tile while the current block's loads are in flight.
struct TileRef {
    int seq, row0, len, tok0;
};
__device__ __forceinline__ TileRef find_tile(const int32_t* __restrict__ cu, const uint32_t* __restrict__ tile_prefix, int32_t n_seqs,
                                             uint32_t t) {
    int lo = 0, hi = n_seqs;
    // when every sequence so far has exactly one tile (batches of merged short sequences), tile t belongs
    // to sequence t: check that before paying for the search
    if ((int)t < n_seqs && tile_prefix[t] <= t && tile_prefix[t + 1] > t) {
        lo = (int)t;
        hi = lo + 1;
    }
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tile_prefix[mid] <= t) lo = mid; else hi = mid;
    }
    while (lo + 1 < n_seqs && tile_prefix[lo + 1] <= t) ++lo;   // skip empty sequences
    TileRef r;
    r.seq = lo;
    r.row0 = (int)(t - tile_prefix[lo]) * kTile;
    r.tok0 = cu[lo];
    r.len = cu[lo + 1] - r.tok0;
    return r;
}

// ---------------------------------------------------------------------------------------------
// Backward helper 1.  For every (128-row tile, head) it writes a [128 rows x 16] bf16 tile holding,
// per query row, -lse/scale (columns 0-2) and -D_i = -sum_c dO_ic O_ic (columns 8-10), each split
// into three bf16 parts whose sum carries 24 bits; the main kernel adds them to its score and dP
// accumulators with a K=16 MMA against a tile of ones.  Rows past the sequence end get -1e30 and 0,
// which makes their probabilities vanish without masking.  The tile is stored in the MMA's shared-
// memory layout (8x8 core matrices; column halves 2048 bytes apart) and is 4 KB-aligned, so one bulk
// copy fetches it.  Also zeroes the fp32 dQ accumulator blocks of sequences longer than one tile (a
// sequence of a single tile gets its dQ written directly by the main kernel).  HBM-bound.
template <int D>
__global__ void __launch_bounds__(256) bwd_pre_kernel(const __nv_bfloat16* __restrict__ o,
                                                      const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ lse,
                                                      const int32_t* __restrict__ cu, const uint32_t* __restrict__ tile_prefix,
                                                      int32_t n_seqs, __nv_bfloat16* __restrict__ stats,
                                                      float* __restrict__ dq_acc, size_t dq_acc_vec4,
                                                      int32_t total_tokens, int32_t n_heads, int32_t head_dim,
                                                      int64_t row_stride, float inv_scale) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_blocks = tile_prefix[n_seqs] * (uint32_t)n_heads;
    for (uint32_t blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
        const uint32_t t = blk / n_heads, h = blk % n_heads;
        // (looking the next block's tile up while this block's loads are in flight, as the post kernel does, made
        // this kernel slower: 0.39 -> 0.44 ms on 131072 tokens x 16 heads)
        const TileRef ref = find_tile(cu, tile_prefix, n_seqs, t);
        const int row0 = ref.row0, len = ref.len, tok0 = ref.tok0;
        if (len > kTile) {
            // this (tile, head) block of the dQ accumulator; a sequence of a single tile needs none (its
            // one tile pair yields the whole dQ, which the main kernel writes directly)
            float4* acc_blk = reinterpret_cast<float4*>(dq_acc) + (size_t)blk * (kTile * D / 4);
            if ((size_t)(blk + 1) * (kTile * D / 4) <= dq_acc_vec4)
                for (int e = threadIdx.x; e < kTile * D / 4; e += blockDim.x) acc_blk[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        {
        uint8_t* out = reinterpret_cast<uint8_t*>(stats) + ((size_t)t * n_heads + h) * (kTile * 16 * 2);
        // Half a warp reads a row with 16-byte loads (D = 128; a quarter warp for D = 64), so that a warp
        // instruction covers 2 (4) rows; a warp takes 16 rows per pass with eight loads of 16 bytes in flight per
        // lane (the kernel waits on HBM latency: bytes in flight are what it runs on).
        constexpr int kLanesPerRow = D / 8;                 // 16 or 8
        constexpr int kRowsPerInst = 32 / kLanesPerRow;     // 2 or 4
        constexpr int kU = 4;                               // row groups in flight per lane
        const int sub = lane / kLanesPerRow, col = (lane % kLanesPerRow) * 8;
        const bool lane_live = col < head_dim;
        const int lane_col = lane_live ? col : 0;
        for (int r0 = warp * kRowsPerInst * kU; r0 < kTile; r0 += 8 * kRowsPerInst * kU) {
            uint4 a[kU], b[kU];
            float nl[kU], acc[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int r = r0 + u * kRowsPerInst + sub;
                a[u] = make_uint4(0u, 0u, 0u, 0u);
                b[u] = make_uint4(0u, 0u, 0u, 0u);
                nl[u] = -1e30f;
                if (row0 + r < len) {
                    const size_t tok = (size_t)tok0 + row0 + r;
                    // rows hold head_dim <= D columns; lanes past them re-read column 0 and drop it, so that the
                    // loads stay unconditional
                    const size_t row = tok * (size_t)row_stride + (size_t)h * head_dim + lane_col;
                    a[u] = *reinterpret_cast<const uint4*>(o + row);
                    b[u] = *reinterpret_cast<const uint4*>(d_o + row);
                    if (!lane_live) a[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (lane % kLanesPerRow == 0) nl[u] = -lse[(size_t)h * total_tokens + tok] * inv_scale;
                }
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w}, bw[4] = {b[u].x, b[u].y, b[u].z, b[u].w};
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[w]));
                    const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[w]));
                    sum += x.x * y.x + x.y * y.y;
                }
#pragma unroll
                for (int sft = kLanesPerRow / 2; sft > 0; sft >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, sft);
                acc[u] = sum;
            }
            // the first lane of a row's group writes its lse chunk, the second its D chunk
            const int role = lane % kLanesPerRow;
            if (role < 2) {
#pragma unroll
                for (int u = 0; u < kU; ++u) {
                    const int r = r0 + u * kRowsPerInst + sub;
                    const float x = role == 0 ? nl[u] : -acc[u];      // every lane of the group holds the row's sum
                    const __nv_bfloat16 b0 = __float2bfloat16(x);
                    const float r1 = x - __bfloat162float(b0);
                    const __nv_bfloat16 b1 = __float2bfloat16(r1);
                    const __nv_bfloat16 b2 = __float2bfloat16(r1 - __bfloat162float(b1));
                    uint4 v;
                    v.x = (uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
                    v.y = (uint32_t)__bfloat16_as_ushort(b2);
                    v.z = 0u;
                    v.w = 0u;
                    *reinterpret_cast<uint4*>(out + role * 2048 + (r / 8) * 128 + (r % 8) * 16) = v;
                }
            }
        }
        }
    }
}

cudaError_t launch_bwd_pre(const __nv_bfloat16* o, const __nv_bfloat16* d_o, const float* lse, const int32_t* cu_seqlens,
                           const SchedView& sched, __nv_bfloat16* stats, float* dq_acc, size_t dq_acc_elems,
                           int32_t total_tokens, int32_t n_heads, int32_t head_dim, int64_t row_stride, float scale,
                           int n_sms, cudaStream_t stream) {
    const int blocks = n_sms * 8;
    if (head_dim > 64)
        bwd_pre_kernel<128><<<blocks, 256, 0, stream>>>(o, d_o, lse, cu_seqlens, sched.tile_prefix, sched.n_seqs, stats,
                                                        dq_acc, dq_acc_elems / 4, total_tokens, n_heads, head_dim,
                                                        row_stride, 1.0f / scale);
    else
        bwd_pre_kernel<64><<<blocks, 256, 0, stream>>>(o, d_o, lse, cu_seqlens, sched.tile_prefix, sched.n_seqs, stats,
                                                       dq_acc, dq_acc_elems / 4, total_tokens, n_heads, head_dim,
                                                       row_stride, 1.0f / scale);
    return cudaGetLastError();
}

// Backward helper 2: dq[T, H, d] = bf16(scale * dq_acc).  dq_acc holds, per (tile, head), a block
// [d/4][128 rows][4 floats]; a CTA reads one block with coalesced 16-byte loads, transposes it in
// shared memory as bf16 and writes whole rows.  Rows past the sequence end are skipped, and so are
// sequences of a single tile, whose dQ the main kernel has already written.
template <int D>
__global__ void __launch_bounds__(256) bwd_post_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq,
                                                       const int32_t* __restrict__ cu, const uint32_t* __restrict__ tile_prefix,
                                                       int32_t n_seqs, int32_t n_heads, int32_t head_dim, int64_t row_stride,
                                                       float scale) {
    constexpr int kRowBytes = D * 2 + 16;                    // padded row of bf16
    __shared__ __align__(16) uint8_t tile[kTile * kRowBytes];
    const uint32_t n_blocks = tile_prefix[n_seqs] * (uint32_t)n_heads;
    if (blockIdx.x >= n_blocks) return;
    TileRef ref = find_tile(cu, tile_prefix, n_seqs, blockIdx.x / n_heads), ref_next = ref;
    for (uint32_t blk = blockIdx.x; blk < n_blocks; blk += gridDim.x, ref = ref_next) {
        const uint32_t t = blk / n_heads, h = blk % n_heads;
        const bool more = blk + gridDim.x < n_blocks;
        const uint32_t t_next = (blk + gridDim.x) / n_heads;
        const int row0 = ref.row0, len = ref.len;
        const int rows = min(kTile, len - row0);
        if (len <= kTile) {               // a single tile pair: the main kernel has written dq itself
            if (more) ref_next = find_tile(cu, tile_prefix, n_seqs, t_next);
            continue;
        }
        const float4* src = reinterpret_cast<const float4*>(dq_acc + ((size_t)t * n_heads + h) * (kTile * D));
        // eight 16-byte loads in flight per thread before the first use (the kernel waits on HBM latency), and the
        // next block's tile is looked up while the first eight are in flight
        for (int e0 = threadIdx.x; e0 < kTile * D / 4; e0 += 8 * 256) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = src[e0 + u * 256];
            if (e0 == (int)threadIdx.x && more) ref_next = find_tile(cu, tile_prefix, n_seqs, t_next);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int e = e0 + u * 256, c4 = e / kTile, r = e % kTile;
                __nv_bfloat162 lo2 = __floats2bfloat162_rn(v[u].x * scale, v[u].y * scale);
                __nv_bfloat162 hi2 = __floats2bfloat162_rn(v[u].z * scale, v[u].w * scale);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo2);
                pk.y = *reinterpret_cast<uint32_t*>(&hi2);
                *reinterpret_cast<uint2*>(tile + r * kRowBytes + c4 * 8) = pk;
            }
        }
        __syncthreads();
        const int kChunks = head_dim * 2 / 16;               // 16-byte chunks per stored row (head_dim <= D columns)
        for (int e = threadIdx.x; e < rows * kChunks; e += blockDim.x) {
            const int r = e / kChunks, c = e % kChunks;
            const uint4 v = *reinterpret_cast<const uint4*>(tile + r * kRowBytes + c * 16);
            __nv_bfloat16* out = dq + ((size_t)ref.tok0 + row0 + r) * (size_t)row_stride + (size_t)h * head_dim;
            reinterpret_cast<uint4*>(out)[c] = v;
        }
        __syncthreads();
    }
}

cudaError_t launch_bwd_post(const float* dq_acc, __nv_bfloat16* dq, const int32_t* cu_seqlens, const SchedView& sched,
                            int32_t n_heads, int32_t head_dim, int64_t row_stride, float scale, int n_sms,
                            cudaStream_t stream) {
    const int blocks = n_sms * 6;
    if (head_dim > 64)
        bwd_post_kernel<128><<<blocks, 256, 0, stream>>>(dq_acc, dq, cu_seqlens, sched.tile_prefix, sched.n_seqs, n_heads,
                                                         head_dim, row_stride, scale);
    else
        bwd_post_kernel<64><<<blocks, 256, 0, stream>>>(dq_acc, dq, cu_seqlens, sched.tile_prefix, sched.n_seqs, n_heads,
                                                        head_dim, row_stride, scale);
    return cudaGetLastError();
}

}  // namespace dcp
