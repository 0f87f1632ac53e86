// Workspace layout and the length-aware work list shared by the forward and backward kernels.
//
// The paper's subject is load imbalance caused by widely varying sequence lengths (Section 2.3);
// on one GPU the same problem shows up as SMs idling while one long sequence finishes.  The work
// list therefore orders sequences longest first, and persistent CTAs pull items from it through a
// global atomic counter, so the cheap items of short sequences fill the tail.
//
// Very short sequences (a 2-D model's temporal axis has 1-13 tokens per sequence) would each
// occupy a whole 128-row tile.  Runs of consecutive short sequences are therefore merged into
// "virtual sequences" of at most 128 tokens that the kernels treat as one tile with a
// block-diagonal mask: the work list is built over the virtual boundaries `vcu` (a subsequence of
// cu_seqlens, padded with empty sequences), and a per-token table gives, for tokens of virtual
// sequences of at most 128 tokens, the range of positions the token's own sequence covers.
#pragma once
#include <cstdint>

namespace dcp {

constexpr int kTile = 128;            // rows of a Q tile / keys of a K,V tile
constexpr int kFwdRowsPerItem = 256;  // a forward work item is two Q tiles of one (sequence, head)
constexpr int kMergeMaxLen = 64;      // sequences longer than this are never merged with their neighbours

// Status codes a kernel may leave in the workspace's status word (0 = no error).
enum : uint32_t {
    kStatusOk = 0,
    kStatusWaitTimeout = 1,
    kStatusBadSmemAlign = 2,
    kStatusBadLengths = 3     // cu_seqlens disagrees with the sizes the caller declared; nothing was computed
};

// First bytes of every workspace.  `status` must stay at offset 0 (dcp_query_status reads it).
// The status word is sticky: kernels only ever raise it (atomicMax), so a failure of any call on this
// workspace stays visible until dcp_query_status has reported and cleared it.  A workspace needs no
// initialisation by the caller: the first kernel of a call that does not find `magic` treats the
// header as fresh memory and clears the status word itself.
constexpr uint32_t kHeaderMagic0 = 0x64637031u, kHeaderMagic1 = 0x9e3779b9u;
constexpr int kMaxCtas = 256;         // persistent CTAs whose time span the header area can record
struct WorkspaceHeader {
    uint32_t status;        // 0 = ok, else the highest kStatus* code a kernel has left since the last query
    uint32_t work_counter;  // next unclaimed work item
    uint32_t n_items;       // items in the list
    uint32_t n_vseq;        // virtual sequences that are not padding
    uint32_t merge_rule;    // which of the two merging rules built them (see merge_kernel)
    uint32_t call_bad;      // this call's boundaries were inconsistent (reset by every call)
    uint32_t magic[2];      // kHeaderMagic0/1 once the header has been initialised
    uint32_t n_ctas[2];     // CTAs of the last forward / backward main launch that recorded a span
    uint32_t pad[54];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is 256 bytes");

#ifdef __CUDACC__
// Run by one thread of the first kernel of every call: a header that does not carry the magic words is
// fresh memory, whose status word means nothing yet.  Afterwards the status word is only ever raised.
__device__ __forceinline__ void header_begin_call(WorkspaceHeader* hdr, bool bad) {
    if (hdr->magic[0] != kHeaderMagic0 || hdr->magic[1] != kHeaderMagic1) {
        hdr->status = kStatusOk;
        hdr->n_ctas[0] = hdr->n_ctas[1] = 0;
        hdr->magic[0] = kHeaderMagic0;
        hdr->magic[1] = kHeaderMagic1;
    }
    hdr->call_bad = bad ? 1u : 0u;
    if (bad) atomicMax(&hdr->status, (uint32_t)kStatusBadLengths);
}
#endif

// When a persistent CTA of the forward (slot 0) or backward main kernel (slot 1) started and when it
// ran out of work, in nanoseconds of the GPU's global timer.  Their spread over the CTAs is the
// single-GPU form of the paper's imbalance ratio (Section 2.3, Section 4.2): with a good work order
// every CTA ends within one item of the others.
struct CtaSpan {
    unsigned long long begin_ns, end_ns;
};
constexpr size_t kSpanBytes = 2 * kMaxCtas * sizeof(CtaSpan);      // 8 KB right after the header

// After the header and the span table: int32 order[n_seqs] (sequence ids, longest first, ties by id),
// uint32 prefix[n_seqs + 1] (items before the i-th sequence of `order`),
// uint32 tile_prefix[n_seqs + 1] (128-row tiles before sequence b, in input order) and
// int32 vcu[n_seqs + 1] (virtual sequence boundaries; unused when sequences are not merged).
// All of these are indexed by VIRTUAL sequence; `cu` is the boundary array the kernels read
// (vcu, or the caller's cu_seqlens when merging is off).
struct SchedView {
    WorkspaceHeader* hdr;
    CtaSpan* spans;         // [2][kMaxCtas]
    const int32_t* order;
    const uint32_t* prefix;
    const uint32_t* tile_prefix;
    const int32_t* vcu;
    int32_t n_seqs;
};

__host__ __device__ constexpr size_t sched_bytes(int32_t n_seqs) {
    return (sizeof(WorkspaceHeader) + kSpanBytes + sizeof(int32_t) * (size_t)n_seqs +
            2 * sizeof(uint32_t) * ((size_t)n_seqs + 1) + sizeof(int32_t) * ((size_t)n_seqs + 1) + 255) & ~(size_t)255;
}

// Per-token table of the merged path: low byte = first position, high byte = one past the last
// position of the token's own sequence, both relative to the start of its virtual sequence.
__host__ __device__ constexpr size_t bounds_bytes(int32_t total_tokens) {
    return (sizeof(uint16_t) * (size_t)total_tokens + 255) & ~(size_t)255;
}

// Upper bound on the number of 128-row tiles of a packed batch: every (virtual) sequence may end in
// a partial tile.  After merging there are at most n_seqs virtual sequences and also at most
// 3 T / 65 + 2: one starts at sequence 0, at a sequence longer than kMergeMaxLen (at most T / 65 of
// those), right after such a sequence, or where the window changes (a window has >= 65 positions).
__host__ __device__ inline size_t max_tiles(int32_t total_tokens, int32_t n_seqs) {
    const size_t by_windows = 3 * ((size_t)total_tokens / (kTile + 1 - kMergeMaxLen)) + 3;
    return (size_t)total_tokens / kTile + ((size_t)n_seqs < by_windows ? (size_t)n_seqs : by_windows);
}

// A decoded work item.  len < 0 marks the end of the list.
struct WorkItem {
    int32_t tok0;   // first token of the sequence in the packed batch
    int32_t len;    // sequence length
    int32_t head;
    int32_t blk;    // row block inside the sequence (256 query rows forward, 128 keys backward)
    int32_t tile0;  // index of the sequence's first 128-row tile among all tiles of the batch
};

// Map item index -> (sequence, head, block).  Within a sequence, blocks vary fastest so that CTAs
// running at the same time share one head's K and V in L2; under a causal mask the heaviest
// blocks come first (forward: last rows see the most keys; backward: first keys are seen by the
// most rows).
__device__ inline WorkItem decode_item(const SchedView& s, const int32_t* cu_seqlens, uint32_t item, int rows_per_blk,
                                       int n_heads, bool heavy_is_last) {
    int lo = 0, hi = s.n_seqs;              // largest i with prefix[i] <= item
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (s.prefix[mid] <= item) lo = mid; else hi = mid;
    }
    const int seq = s.order[lo];
    WorkItem w;
    w.tok0 = cu_seqlens[seq];
    w.len = cu_seqlens[seq + 1] - w.tok0;
    w.tile0 = (int32_t)s.tile_prefix[seq];
    const uint32_t local = item - s.prefix[lo];
    const uint32_t nblk = (uint32_t)(w.len + rows_per_blk - 1) / (uint32_t)rows_per_blk;
    w.head = (int32_t)(local / nblk);
    const uint32_t b = local % nblk;
    w.blk = (int32_t)(heavy_is_last ? nblk - 1 - b : b);
    (void)n_heads;
    return w;
}

}  // namespace dcp
