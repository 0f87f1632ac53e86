// Host-visible launch interface of the attention kernels (internal to libdcp).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "sched.cuh"

namespace dcp {

struct FwdParams {
    const int32_t* cu_seqlens;    // boundaries of the (virtual) sequences the work list was built over
    const uint16_t* bounds;       // per-token table of the merged path (see sched.cuh), or null
    __nv_bfloat16* o;
    float* lse;
    SchedView sched;
    int32_t n_heads;
    int32_t head_dim;     // columns of a row in global memory (a multiple of 8); the kernels work on 64 or 128
                          // columns, those past head_dim read as zeros (TMA fills them) and are never stored
    int32_t total_tokens;
    int64_t row_stride; // elements between consecutive tokens of q, k, v, o (n_heads * head_dim when contiguous)
    float scale;        // softmax scale
    float scale_log2;   // scale * log2(e)
};

struct BwdParams {
    const int32_t* cu_seqlens;    // as in FwdParams
    const uint16_t* bounds;
    const __nv_bfloat16* stats;   // per (tile, head) a [128 queries x 16] bf16 tile in the layout the MMA reads:
                                  // columns 0-2 = -lse/scale split in three bf16 parts, 8-10 = -D likewise
                                  // (D_i = sum_c dO_ic O_ic); rows past the sequence end hold -1e30 and 0
    float* dq_acc;        // fp32, tile-blocked: [tile][head][d/4][128 rows][4]; zeroed before the main kernel
    __nv_bfloat16* dq;    // final dQ: written directly for sequences of a single tile, by the post kernel otherwise
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    SchedView sched;
    int32_t n_heads;
    int32_t head_dim;     // as in FwdParams
    int32_t total_tokens;
    int64_t row_stride;   // as in FwdParams; the same for q, k, v, dO, dq, dk, dv
    float scale;
    float scale_log2;
};

// Builds the work list (longest sequence first) and resets the work counter and status word.
// With `bounds` non-null, short sequences are first merged into virtual sequences: sched.vcu and
// `bounds` are written and the list is built over sched.vcu, which the later kernels must then be
// given as their boundary array; with `bounds` null the list is built over cu_seqlens itself.
int prep_launches(int32_t n_seqs, bool merge, bool input_order);   // kernels launch_prep enqueues (1 to 4)
// tile_capacity = number of 128-row tiles the per-tile storage of the workspace holds (UINT32_MAX if the
// call uses none).  Inconsistent boundaries or more tiles than that leave an empty work list and
// kStatusBadLengths in the status word.  input_order = true lists the sequences as they come instead of
// longest first (a measurement aid: it shows what the ordering is worth).
cudaError_t launch_prep(const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen,
                        int32_t rows_per_block, int32_t n_heads, const SchedView& sched, uint16_t* bounds,
                        uint32_t tile_capacity, bool input_order, cudaStream_t stream);

// One CTA that waits, with the kernels' own bounded wait and the given poll limit, on a barrier nobody
// arrives at, and leaves through the same abort path (status word raised, no trap).
cudaError_t launch_wait_timeout_selftest(WorkspaceHeader* hdr, uint32_t spin_limit, cudaStream_t stream);

// Copies row ranges between two tensors (see dcp_copy_segments).
cudaError_t launch_copy_segments(const void* src, void* dst, const int32_t* seg, int32_t n_seg, int64_t row_bytes,
                                 int32_t n_planes, int64_t src_plane_bytes, int64_t dst_plane_bytes, bool reverse,
                                 int n_sms, cudaStream_t stream);

// short_items: no sequence of the batch is longer than a few dozen tiles, so work items are short and the
// variant that releases Q slots early pays (under a causal mask it always does).
// `to` = the same kind of map over o: whole tiles leave through shared memory and TMA stores.
cudaError_t launch_attn_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                            const FwdParams& p, int head_dim, bool causal, bool short_items, int n_ctas, cudaStream_t stream);

// Tile-aligned row statistics for the backward kernel (see BwdParams::stats) and dq_acc = 0.
cudaError_t launch_bwd_pre(const __nv_bfloat16* o, const __nv_bfloat16* d_o, const float* lse, const int32_t* cu_seqlens,
                           const SchedView& sched, __nv_bfloat16* stats, float* dq_acc, size_t dq_acc_elems,
                           int32_t total_tokens, int32_t n_heads, int32_t head_dim, int64_t row_stride, float scale,
                           int n_sms, cudaStream_t stream);

// tdk, tdv = maps over dk and dv: whole key blocks leave through shared memory and TMA stores.
cudaError_t launch_attn_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                            const CUtensorMap& tdk, const CUtensorMap& tdv, const BwdParams& p, int head_dim, bool causal,
                            int n_ctas, cudaStream_t stream);

// dq[T, H, d] = bf16(scale * dq_acc), undoing the tile-blocked layout
cudaError_t launch_bwd_post(const float* dq_acc, __nv_bfloat16* dq, const int32_t* cu_seqlens, const SchedView& sched,
                            int32_t n_heads, int32_t head_dim, int64_t row_stride, float scale, int n_sms,
                            cudaStream_t stream);

// Batches in which no sequence exceeds kSmallSeqMaxLen tokens (the declared max_seqlen says so) skip the work list
// and the 128-row tile kernels, see attn_small.cu.  The check kernel is the first of such a call (boundaries
// consistent, no sequence longer than declared; it also fills first_seq, 2 n_seqs + 1 entries of scratch); the
// attention kernel computes nothing if it found a fault.  The backward does not read `o`.
constexpr int kSmallSeqMaxLen = 32;
bool small_path_fits(int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen);
cudaError_t launch_small_check(bool backward, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen,
                               int32_t n_heads, WorkspaceHeader* hdr, int32_t* first_seq, int n_sms, cudaStream_t stream);
// forward: o and lse written (d_o, dq, dk, dv null); backward: lse read, dq, dk, dv written (o null)
cudaError_t launch_small_attn(bool backward, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* d_o, float* lse, const int32_t* cu_seqlens, int32_t total_tokens,
                              int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int64_t row_stride, bool causal, float scale,
                              __nv_bfloat16* o, __nv_bfloat16* dq, __nv_bfloat16* dk, __nv_bfloat16* dv, WorkspaceHeader* hdr,
                              const int32_t* first_seq, int n_sms, cudaStream_t stream);

}  // namespace dcp
