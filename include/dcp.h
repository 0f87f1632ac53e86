/*
 * dcp.h - C ABI of the B200 (sm_100a) packed variable-length attention library and of the
 * single-GPU micro-batch / recomputation planner.
 *
 * All entry points return an int status (DCP_OK = 0).  No exception crosses this boundary and no
 * entry point below allocates device memory: every buffer, the workspace included, belongs to the
 * caller.  On any error the outputs are left untouched and dcp_last_error() gives a message.
 *
 * Tensor layout: q, k, v, o, d_o, dq, dk, dv are bf16, shape [total_tokens, n_heads, head_dim],
 * contiguous, sequences packed back to back; sequence b owns tokens cu_seqlens[b] ..
 * cu_seqlens[b+1]-1.  lse is fp32, shape [n_heads, total_tokens].  Device pointers must be
 * 16-byte aligned.  Supported head_dim: multiples of 8 up to 128 (64 and 128 are native; the
 * others run zero-padded to the next of the two).  n_heads is the same for q, k and v.
 */
#ifndef DCP_H_
#define DCP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    DCP_OK = 0,
    DCP_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer, ...            */
    DCP_ERR_INFEASIBLE = 2,  /* planner: one sequence exceeds the budget even at full recompute */
    DCP_ERR_UNSUPPORTED = 3, /* head_dim not a multiple of 8 up to 128, device is not sm_100    */
    DCP_ERR_WORKSPACE = 4,   /* workspace missing or smaller than dcp_varlen_attn_workspace     */
    DCP_ERR_CUDA = 5,        /* a CUDA runtime/driver call or a launch failed                   */
    DCP_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (see dcp_query_status)       */
    DCP_ERR_OVERFLOW = 7     /* planner: a quantity does not fit in int64                       */
};

/* ---------------------------------------------------------------------------------------------
 * Planner.
 *
 * Paper: Section 3.2 (problem statement; here at sequence-parallel size p = 1, so only the
 * throughput target Eq. 1 remains), Section 3.4 Eq. 4-6 (time and memory of a batch with r
 * recomputed layers) and the inner rule of Algorithm 1 (smallest recompute count that fits the
 * memory capacity); Section 3.1 (sequences of similar length are grouped).
 *
 * Splits one batch of sequences into gradient-accumulation micro-batches and picks, per
 * micro-batch, how many layers recompute their forward pass, minimising modelled time under an
 * HBM budget.  Indices are sorted by (length descending, index ascending); a plan is a split of
 * that order into contiguous blocks.  For a block with tok = sum L and W = sum L^2:
 *     m = 4*tok*H*d*e,  m_inp = tok*H*d*e,  mem(r) = (Lambda-r)*m + Lambda*m_inp + M_C,
 *     r* = smallest r in [0, Lambda] with mem(r) <= budget,
 *     time = Lambda*7*W + r* * 2*W + T_C.
 * Returned cost = K*T_C + 2*sum_k r*_k W_k (the plan-independent part is dropped).  Ties: fewer
 * micro-batches, then the lexicographically largest block-size vector.
 * Host pointers throughout; runs on the host only; integer arithmetic only (int64, checked).
 */
typedef struct {
    int32_t n_heads;     /* H, >= 1 */
    int32_t head_dim;    /* d, >= 1 */
    int32_t elt_bytes;   /* e, >= 1 (2 for bf16) */
    int32_t n_layers;    /* Lambda, >= 1; with 1 the recompute count is a 0/1 flag */
    int64_t const_bytes; /* M_C >= 0 */
    int64_t fixed_cost;  /* T_C >= 0, in units of one L^2 product over all heads */
} dcp_plan_params;

/* params == NULL selects H = 16, d = 128, e = 2, Lambda = 1, M_C = 0, T_C = 2^24.
 * lengths [n] (each >= 1), n >= 1.  Outputs: mb_id [n] = micro-batch of each INPUT index
 * (micro-batch 0 holds the longest sequence); *n_mb = K; recompute [n], first K entries valid;
 * cost (nullable). */
int dcp_plan(const int32_t* lengths, int32_t n, int64_t hbm_budget_bytes, const dcp_plan_params* params,
             int32_t* mb_id, int32_t* n_mb, int32_t* recompute, int64_t* cost);

/* The same planner fed by profiled times instead of the L^2 model.
 *
 * Paper: Section 3.5 (dual-layer profiling: the forward time t_f of one layer is measured per
 * candidate and the whole model is extrapolated from it) and Eq. 5 (recomputing r layers costs
 * r * t_f).  fwd_time [n] (host, each >= 0) is the measured or interpolated per-layer forward time
 * of sequence i in any integer unit (nanoseconds, say); T_C (params->fixed_cost) is in the same
 * unit.  Memory model, ordering, tie rules, outputs and errors are those of dcp_plan; the cost is
 * K*T_C + sum_k r*_k * sum_{i in block k} fwd_time[i].  With fwd_time[i] = 2 * lengths[i]^2 the
 * result equals dcp_plan's. */
int dcp_plan_profiled(const int32_t* lengths, const int64_t* fwd_time, int32_t n, int64_t hbm_budget_bytes,
                      const dcp_plan_params* params, int32_t* mb_id, int32_t* n_mb, int32_t* recompute,
                      int64_t* cost);

/* DCP-intra: batch size, sequence-parallel size and recompute count for one sequence length.
 *
 * Paper: Section 3.4, Eq. 4-6 and Algorithm 1.  Each candidate (b, p) carries what the dual-layer
 * profile (Section 3.5) gives with EVERY layer recomputed: the forward time t_f of one layer, the
 * activation bytes m one layer keeps when it is not recomputed, the iteration time T_(b,p) and the
 * memory M_(b,p).  Letting `keep` layers keep their activations costs keep*m bytes and saves
 * keep*t_f, so per candidate keep = min(Lambda, floor((capacity - M_(b,p)) / m)), the recompute count
 * is r = Lambda - keep (the smallest that fits) and the time T_(b,p) - keep*t_f.  The listing's loop
 * stops at the first count that fits; it is read as "the largest count that still fits", which is
 * what its comment and the text say.  Among candidates the one with the highest throughput
 * b / (p * time) wins (Eq. 1; the text says throughput, the listing compares times, which is the
 * same when b and p are equal).  Ties: smaller p, then larger b, then the earlier candidate.
 * Candidates with M_(b,p) > capacity are skipped; none left => DCP_ERR_INFEASIBLE.
 * Host pointers; outputs *best (index), *recompute (r), time (nullable).  On one GPU every p is 1;
 * the function itself does not touch a device. */
typedef struct {
    int32_t batch_size; /* b >= 1 */
    int32_t sp_size;    /* p >= 1 */
    int64_t t_f;        /* >= 0, any integer time unit */
    int64_t m;          /* >= 0, bytes */
    int64_t time_full;  /* T_(b,p) >= 1, same unit as t_f */
    int64_t mem_full;   /* M_(b,p) >= 0, bytes */
} dcp_intra_candidate;

int dcp_intra_select(const dcp_intra_candidate* cands, int32_t n, int64_t mem_capacity, int32_t n_layers,
                     int32_t* best, int32_t* recompute, int64_t* time);

/* DCP-inter: accumulation-step counts that balance n batches running side by side.
 *
 * Paper: Section 3.3, Eq. 3, and Appendix C (G_min, G_max).  Batch i takes times[i] (any positive
 * integer unit: modelled cost, measured microseconds) per accumulation step on its worker group.
 * Chooses g[i] >= 1 minimising the idle time sum_i (max_j g_j T_j - g_i T_i) subject to
 * g_i T_i <= G_max * max_j T_j.  Ties: shorter iteration max_j g_j T_j, then the lexicographically
 * smallest g.  Afterwards, if max_i g_i < G_min, every g_i is multiplied by ceil(G_min / max_i g_i).
 * On a single GPU this is a planning/simulation aid (the n worker groups are virtual); nothing here
 * touches the device.  Host pointers; outputs g [n], idle and iteration_time (both nullable, after
 * the G_min scaling).  Errors: DCP_ERR_INVALID_ARG, DCP_ERR_OVERFLOW, DCP_ERR_UNSUPPORTED (more than
 * 4e6 candidate iteration times, i.e. times differing by many orders of magnitude). */
int dcp_inter_plan(const int64_t* times, int32_t n, int32_t g_min, int32_t g_max, int32_t* g, int64_t* idle,
                   int64_t* iteration_time);

/* ---------------------------------------------------------------------------------------------
 * Attention.
 *
 * Paper: Section 4.1 ("Implementation details": a fused attention library is enabled in every
 * run) and Section 4.2 ("Effect of model architecture": attention time dominates).  The paper
 * gives no formula; the operation is softmax(Q K^T * scale + mask) V per sequence and head, with
 * key j visible to query i iff (not causal) or j <= i, indices relative to the sequence start.
 * lse_i = ln sum_j exp(scale * q_i.k_j) over visible keys (natural log).
 *
 * Both calls only enqueue work on `cuda_stream` (a cudaStream_t; NULL = the default stream);
 * they neither synchronise nor read cu_seqlens on the host.  softmax_scale = 0 selects
 * 1/sqrt(head_dim).  Zero-length sequences are legal.  max_seqlen must be >= every length.
 * cu_seqlens is checked on the device (it must start at 0, never decrease, end at total_tokens, and
 * fit the workspace that max_seqlen promised): if it does not hold, the call computes nothing,
 * leaves the outputs as they were and dcp_query_status returns DCP_ERR_INVALID_ARG.
 */

/* Bytes of caller-provided device workspace needed by the forward and the backward call: the work
 * list (per sequence), a 2-byte-per-token table used when runs of short sequences share a tile, and for
 * the backward the per-row statistics and the fp32 dQ accumulator (per 128-row tile and head). */
int dcp_varlen_attn_workspace(int32_t total_tokens, int32_t n_seqs, int32_t n_heads, int32_t head_dim,
                              size_t* fwd_bytes, size_t* bwd_bytes);

/* q, k, v (device, in) -> o, lse (device, out).  workspace: device, >= fwd_bytes, 256-byte
 * aligned; its first word is a status word that dcp_query_status reads. */
int dcp_varlen_attn_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens, int32_t n_seqs,
                        int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                        int32_t causal, float softmax_scale, void* o, float* lse, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* Gradients of sum(o * d_o): q, k, v, o, d_o, lse (device, in) -> dq, dk, dv (device, out).
 * `causal` and `softmax_scale` must equal the forward call's.  workspace >= bwd_bytes; it holds
 * the fp32 dQ accumulator and the per-row D = sum_c dO*O.  dQ is summed with floating-point
 * atomics, so its low bits may differ from run to run. */
int dcp_varlen_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                        const float* lse, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                        int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int32_t causal,
                        float softmax_scale, void* dq, void* dk, void* dv, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* Forward attention without a workspace argument (the paper has no counterpart; this exists for
 * callers that must not allocate device memory - code running inside a memory-pool callback or a
 * real-time loop, a plug-in handed fixed buffers by its host program, a process whose allocator is
 * locked down after start-up).  Same operation, arguments, layouts and error codes as
 * dcp_varlen_attn_fwd, but the work-list scratch is a fixed array inside the library's device
 * image (about 66 KB, held by every GPU that loads the library until the process exits) instead of
 * a caller buffer.  Limits and rules:
 *   - runs of very short sequences are not merged into shared tiles here (the table that needs grows
 *     with the token count), so such batches run slower than through dcp_varlen_attn_fwd; results
 *     agree within rounding (sequences of at most 128 tokens take different code paths);
 *   - n_seqs <= DCP_NOALLOC_MAX_SEQS, else DCP_ERR_UNSUPPORTED and nothing is enqueued;
 *   - the call allocates nothing on the device and frees nothing;
 *   - the first call on each device looks up the array's device address (a synchronous runtime
 *     query); make that first call before starting any stream capture on that device;
 *   - all calls on a device share the one array, which keeps the previous call's contents; the
 *     library re-initialises what it needs at the start of every call, but two calls whose kernels
 *     may overlap on the GPU (different streams) race on it - serialise them;
 *   - the device status word of this variant lives in that array and is not readable through
 *     dcp_query_status; the kernels' waits are bounded all the same. */
#define DCP_NOALLOC_MAX_SEQS 4096
int dcp_varlen_attn_fwd_noalloc(const void* q, const void* k, const void* v, const int32_t* cu_seqlens, int32_t n_seqs,
                                int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                                int32_t causal, float softmax_scale, void* o, float* lse, void* cuda_stream);

/* Synchronises `cuda_stream`, then reads the status word at the start of `workspace`.
 * Returns DCP_OK, DCP_ERR_TIMEOUT (a kernel abandoned a bounded wait; results are invalid),
 * DCP_ERR_INVALID_ARG (cu_seqlens was inconsistent; nothing was computed) or DCP_ERR_CUDA. */
int dcp_query_status(const void* workspace, void* cuda_stream);

/* Measurement aid (no counterpart in the paper).  While enabled, every attention call records a
 * pair of CUDA events around each kernel it launches, on the caller's stream.  dcp_profile_read
 * waits for those events, adds up device time (ms) and launch counts per kernel since the previous
 * read into ms[DCP_N_KERNELS] and launches[DCP_N_KERNELS] (host pointers), and forgets them. */
enum {
    DCP_KERNEL_PREP = 0,     /* work-list construction            */
    DCP_KERNEL_FWD = 1,      /* forward attention                 */
    DCP_KERNEL_BWD_PRE = 2,  /* D = rowsum(dO*O), zero dQ accum.  */
    DCP_KERNEL_BWD_MAIN = 3, /* backward attention                */
    DCP_KERNEL_BWD_POST = 4, /* dQ fp32 -> bf16                   */
    DCP_N_KERNELS = 5
};
int dcp_profile_enable(int on);
int dcp_profile_read(float* ms, int64_t* launches);

/* Number of kernel launches this library has enqueued since it was loaded (all threads). */
int64_t dcp_launch_count(void);

/* Message for the last error on the calling thread ("" if none). The pointer stays valid until
 * the thread's next failing call. */
const char* dcp_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DCP_H_ */
