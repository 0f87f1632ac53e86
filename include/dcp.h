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

/* A candidate of dcp_intra_select (described there). */
typedef struct {
    int32_t batch_size; /* b >= 1 */
    int32_t sp_size;    /* p >= 1 */
    int64_t t_f;        /* >= 0, any integer time unit */
    int64_t m;          /* >= 0, bytes */
    int64_t time_full;  /* T_(b,p) >= 1, same unit as t_f */
    int64_t mem_full;   /* M_(b,p) >= 0, bytes */
} dcp_intra_candidate;

/* Data layout of a planned batch.
 *
 * Paper: Section 3.1 (the settings chosen for an incoming batch are applied to that batch's data:
 * its sequences are regrouped into the micro-batches the plan names).  The batch's tensors hold the
 * sequences packed in input order; micro-batch k gets its own packed tensors holding, in input
 * order, the sequences i with mb_id[i] == k.  This call turns (lengths, mb_id) into what the copies
 * and the attention calls need.  Host pointers; nothing touches a device.  Outputs:
 *   mb_seq_offset [n_mb + 1]  micro-batch k owns entries mb_seq_offset[k] .. mb_seq_offset[k+1]-1 of seq_index
 *   seq_index [n]             input index of every entry
 *   mb_cu [n + n_mb]          micro-batch k's boundary array (its cu_seqlens, starting at 0) occupies
 *                             mb_cu[mb_seq_offset[k] + k ...], one entry more than it has sequences
 *   seg_offset [n_mb + 1], seg [3 * seg_capacity], *n_seg
 *                             micro-batch k's copy list is seg[3*seg_offset[k] .. 3*seg_offset[k+1]): triples
 *                             (first row in the batch, first row in the micro-batch, rows), each at most
 *                             max_rows rows (long sequences are cut so that a copy kernel's CTAs get
 *                             pieces of similar size) - the form dcp_copy_segments takes.
 * lengths may contain zeros.  If seg_capacity is too small the call returns DCP_ERR_WORKSPACE with
 * *n_seg set to the number needed (n + sum(lengths) / max_rows always suffices). */
int dcp_plan_segments(const int32_t* lengths, const int32_t* mb_id, int32_t n, int32_t n_mb, int32_t max_rows,
                      int32_t* mb_seq_offset, int32_t* seq_index, int32_t* mb_cu, int32_t* seg_offset, int32_t* seg,
                      int32_t seg_capacity, int32_t* n_seg);

/* Copies row ranges between two device tensors on `cuda_stream` (enqueue only): the gather of a
 * micro-batch's sequences out of a batch and the scatter of its results back (Section 3.1, as above).
 * seg: device int32 [n_seg][3] = (a, b, rows).  reverse == 0: rows b.. of dst = rows a.. of src;
 * reverse != 0: rows a.. of dst = rows b.. of src.  A row is row_bytes bytes (a multiple of 4; 16-byte
 * multiples with 16-byte aligned tensors take the fast path).  n_planes > 1 repeats the copy for planes
 * src_plane_bytes / dst_plane_bytes apart: lse [n_heads, T] is n_heads planes of 4-byte rows.  Ranges
 * must lie inside both tensors and must not overlap in dst; nothing checks that. */
int dcp_copy_segments(const void* src, void* dst, const int32_t* seg, int32_t n_seg, int64_t row_bytes,
                      int32_t n_planes, int64_t src_plane_bytes, int64_t dst_plane_bytes, int32_t reverse,
                      void* cuda_stream);

/* Profiled times between the profiled lengths.
 *
 * Paper: Section 3.5 measures t_f, t_b per candidate; it does not say how a length between two
 * profiled ones is handled.  Here: bucket_len [n_buckets] strictly ascending, bucket_val the measured
 * per-sequence value (any integer unit, >= 0).  For a length L: below the first bucket linear in L
 * (val_0 * L / len_0: short sequences are bound by memory traffic); between two buckets linear; above
 * the last quadratic (val_last * L^2 / len_last^2: attention time).  Floor division throughout.
 * Host pointers; out [n]. */
int dcp_profile_interp(const int32_t* bucket_len, const int64_t* bucket_val, int32_t n_buckets, const int32_t* lengths,
                       int32_t n, int64_t* out);

/* Modelled time of one micro-batch, Eq. 4-5: Lambda * (sum t_f + sum t_b) + r * sum t_f + T_C, from
 * the per-sequence per-layer times fwd_time, bwd_time [n] (host). */
int dcp_model_time(const int64_t* fwd_time, const int64_t* bwd_time, int32_t n, int32_t n_layers, int32_t recompute,
                   int64_t fixed_cost, int64_t* time);

/* One row of the candidate table Algorithm 1 takes, from a dual-layer measurement (Section 3.5: the
 * profile runs with every layer recomputed and the model is extrapolated as
 * T_(b,p) = Lambda * (2 t_f + t_b) + T_C; Eq. 6 at r = Lambda gives M_(b,p) = Lambda * m_inp + M_C).
 * t_f, t_b: measured forward / backward time of one layer for the whole candidate batch; act_bytes = m,
 * what one layer keeps when it is not recomputed; inp_bytes = m_inp. */
int dcp_intra_candidate_from_profile(int32_t batch_size, int32_t sp_size, int64_t t_f, int64_t t_b, int64_t act_bytes,
                                     int64_t inp_bytes, int32_t n_layers, int64_t const_bytes, int64_t fixed_cost,
                                     dcp_intra_candidate* out);

/* The planner's memory model for `tokens` tokens of one micro-batch (Eq. 6 with the sizes this build's
 * benchmark fixes): a layer that is not recomputed keeps act_bytes = m = 4 * tokens * H * d * e (q, k, v, o),
 * every layer keeps its input, inp_bytes = m_inp = tokens * H * d * e.  Host pointers. */
int dcp_activation_bytes(int64_t tokens, int32_t n_heads, int32_t head_dim, int32_t elt_bytes, int64_t* act_bytes,
                         int64_t* inp_bytes);

/* Micro-batches of a group of n_seqs sequences of one length run with the batch size Algorithm 1 selected
 * for that length (Section 3.4): consecutive sequences share a micro-batch, mb_id [n_seqs] (host) = i / b,
 * *n_mb = ceil(n_seqs / b).  Feed mb_id to dcp_plan_segments. */
int dcp_length_group_plan(int32_t n_seqs, int32_t batch_size, int32_t* mb_id, int32_t* n_mb);

/* Which rank owns which sequence when a batch is sharded over world_size GPUs without any
 * data-path collective (every (sequence, head) is independent).
 *
 * Paper: Section 2.3 (imbalance across devices comes from sequence length; attention cost grows with
 * L^2).  Sequences are dealt longest first (ties by index) to the rank with the least accumulated
 * L^2 (lowest rank on ties).  Host pointers; rank_of [n]; load [world_size] (nullable) = sum of L^2. */
int dcp_shard_sequences(const int32_t* lengths, int32_t n, int32_t world_size, int32_t* rank_of, int64_t* load);

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
 * The workspace needs no initialisation and may be reused by any number of calls on one stream.
 */

/* Bytes of caller-provided device workspace needed by the forward and the backward call: the work
 * list (per sequence), a 2-byte-per-token table used when runs of short sequences share a tile, and for
 * the backward the per-row statistics and the fp32 dQ accumulator (per 128-row tile and head). */
int dcp_varlen_attn_workspace(int32_t total_tokens, int32_t n_seqs, int32_t n_heads, int32_t head_dim,
                              size_t* fwd_bytes, size_t* bwd_bytes);

/* q, k, v (device, in) -> o, lse (device, out).  workspace: device, >= fwd_bytes, 256-byte
 * aligned; its first word is a status word that dcp_query_status reads and clears. */
int dcp_varlen_attn_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens, int32_t n_seqs,
                        int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                        int32_t causal, float softmax_scale, void* o, float* lse, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* Gradients of sum(o * d_o): q, k, v, o, d_o, lse (device, in) -> dq, dk, dv (device, out).
 * `causal` and `softmax_scale` must equal the forward call's.  workspace >= bwd_bytes; it holds
 * the fp32 dQ accumulator and the per-row D = sum_c dO*O.  dQ is summed with floating-point
 * atomics, so its low bits may differ from run to run.  When max_seqlen <= 32 (see
 * dcp_set_short_sequence_path) D is formed as sum_j P_ij dP_ij instead, `o` is not read, and the
 * result is the same from run to run. */
int dcp_varlen_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                        const float* lse, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                        int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int32_t causal,
                        float softmax_scale, void* dq, void* dk, void* dv, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* The same two calls on a group of heads inside wider tensors: consecutive tokens of q, k, v, o, d_o, dq,
 * dk, dv are token_stride elements apart (a multiple of 8, at least n_heads * head_dim; the plain calls are
 * the case token_stride = n_heads * head_dim); each pointer addresses the group's first head of token 0; lse
 * stays [n_heads, total_tokens] for the group.
 *
 * Paper: Section 3.2 (sequence-parallel size p_i) and Section 4.1 (the head-sharded scheme: every rank of
 * a group holds a slice of the tokens with all heads, attention needs all tokens of some heads).  With these
 * calls rank r of p computes heads [r H/p, (r+1) H/p) directly on the token-sharded [T, H, d] tensors - its
 * own slice and its peers', mapped into one address range (peer or fabric mappings; the kernels read them
 * with plain TMA loads, no multicast, and write results with plain stores) - so the re-sharding all-to-all
 * on either side of attention is never materialised: a tile crosses the link when the kernel needs it. */
int dcp_varlen_attn_fwd_strided(const void* q, const void* k, const void* v, const int32_t* cu_seqlens, int32_t n_seqs,
                                int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                                int64_t token_stride, int32_t causal, float softmax_scale, void* o, float* lse,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);
int dcp_varlen_attn_bwd_strided(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                const float* lse, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens,
                                int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int64_t token_stride,
                                int32_t causal, float softmax_scale, void* dq, void* dk, void* dv, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/* Forward attention without a workspace argument (the paper has no counterpart; this exists for
 * callers that must not allocate device memory - code running inside a memory-pool callback or a
 * real-time loop, a plug-in handed fixed buffers by its host program, a process whose allocator is
 * locked down after start-up).  Same operation, arguments, layouts and error codes as
 * dcp_varlen_attn_fwd, but the work-list scratch is a fixed array inside the library's device
 * image (about 74 KB, held by every GPU that loads the library until the process exits) instead of
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
 *   - the device status word of this variant lives in that array: dcp_noalloc_status reads it. */
#define DCP_NOALLOC_MAX_SEQS 4096
int dcp_varlen_attn_fwd_noalloc(const void* q, const void* k, const void* v, const int32_t* cu_seqlens, int32_t n_seqs,
                                int32_t total_tokens, int32_t max_seqlen, int32_t n_heads, int32_t head_dim,
                                int32_t causal, float softmax_scale, void* o, float* lse, void* cuda_stream);

/* dcp_query_status for the built-in array of dcp_varlen_attn_fwd_noalloc on the current device
 * (synchronises `cuda_stream`, reports and clears).  It allocates nothing either. */
int dcp_noalloc_status(void* cuda_stream);

/* Synchronises `cuda_stream`, then reads the status word at the start of `workspace`.  The word is
 * sticky on the device: it keeps the most severe failure of ANY call made on this workspace since the
 * previous query, and this call clears it after reporting.
 * Returns DCP_OK, DCP_ERR_TIMEOUT (a kernel abandoned a bounded wait; results are invalid),
 * DCP_ERR_INVALID_ARG (cu_seqlens was inconsistent; that call computed nothing) or DCP_ERR_CUDA. */
int dcp_query_status(void* workspace, void* cuda_stream);

/* Self-test of the bounded-wait path (no counterpart in the paper).  Every device-side wait of this
 * library gives up after a poll limit, raises the workspace's status word and lets its CTA run to the
 * end instead of hanging the GPU.  This call enqueues one tiny CTA that waits, with that same helper and
 * a limit of `spin_limit` polls (at most 2^20), on a barrier nothing ever arrives at, and then returns
 * normally; dcp_query_status(workspace) must afterwards report DCP_ERR_TIMEOUT.  It never traps.
 * workspace: device, at least 256 bytes, 256-byte aligned. */
int dcp_selftest_wait_timeout(void* workspace, uint32_t spin_limit, void* cuda_stream);

/* Measurement aids for the work order (no counterpart in the paper beyond the problem itself:
 * Section 2.3's imbalance, which on one GPU shows as SMs idling while one long sequence finishes).
 * dcp_set_work_order(1) makes later calls list sequences as they come instead of longest first;
 * dcp_set_work_order(0) restores the default.  Process-wide.
 * dcp_read_cta_spans synchronises `cuda_stream` and returns, for the last forward (which = 0) or
 * backward main (which = 1) launch on `workspace`, when each persistent CTA started and when it ran
 * out of work, in nanoseconds of the GPU's global timer: begin_ns, end_ns [256] (host), *n_ctas valid. */
int dcp_set_work_order(int input_order);

/* Batches of very short sequences (Section 4.1: the temporal axis of a 2-D model has sequences of a handful
 * of tokens).  When the declared max_seqlen is at most 32, dcp_varlen_attn_fwd/bwd (and their strided and
 * no-allocation forms) run one small CTA per (sequence, group of heads) that fetches exactly the sequence's
 * rows, instead of the work list and the 128-row tile kernels: such a batch is bound by HBM, and what it needs
 * is many sequences in flight per SM.  Results are the same within rounding; the backward then forms
 * D_i = sum_j P_ij dP_ij itself and does not read `o`; a sequence longer than the declared max_seqlen makes
 * dcp_query_status report DCP_ERR_INVALID_ARG and nothing is computed (as on the other path).
 * dcp_set_short_sequence_path(0) sends such batches through the tile kernels instead (a measurement aid and
 * a test hook); 1 restores the default.  Process-wide. */
int dcp_set_short_sequence_path(int enabled);
int dcp_read_cta_spans(const void* workspace, int32_t which, void* cuda_stream, int64_t* begin_ns, int64_t* end_ns,
                       int32_t* n_ctas);

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
