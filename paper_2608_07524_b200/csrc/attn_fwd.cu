// Forward packed variable-length attention for sm_100a.
//
// One persistent CTA per SM.  A work item is (sequence, head, 256 query rows) = two 128-row Q
// tiles.  Roles:
//   warps 0-3   softmax group 0 (Q tile 0): one thread per query row
//   warps 4-7   softmax group 1 (Q tile 1)
//   warp  8     MMA issue (one thread): S_t = Q_t K_j^T and O_t += P_t V_j with tcgen05, fp32
//               accumulators in tensor memory
//   warp  9     scheduler + TMA producer (one thread): pulls work items from the global counter,
//               streams Q once and K_j, V_j through a shared-memory ring
//   warps 10-11 idle; they exist so that warps 8-11 form a group that can hand its registers to
//               the softmax groups (setmaxnreg), which hold a whole 128-wide score row per thread
// The two Q tiles alternate on the tensor pipe: while one group runs exp on its S tile, the pipe
// computes the other tile's products.  P overwrites S in tensor memory as packed bf16 and is the
// A operand of the second product, so probabilities never touch shared memory.
//
// Softmax is the online form: a running row maximum m and sum l; the maximum is only raised when
// it grew by more than 2^8, which keeps exp2 arguments bounded while making rescales of the O
// accumulator rare.  Results: O = acc / l (bf16), lse = m*scale + ln l (fp32).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sched.cuh"
#include "sm100_ptx.cuh"

namespace dcp {

// One pair of exponentials in this many is computed on the FMA pipe instead of the special-function
// unit (0: none).  Measured on the forward kernel alone: bidirectional config 3, 18.2 ms with none,
// 17.8 with packed arithmetic only, 17.5 / 17.1 / 17.1 with every 8th / 4th / 3rd pair, 18.7 with every
// 2nd; causal config 2, 1.23 / 1.17 / 1.17 / 1.23 / 1.23 ms.
constexpr int kPolyEveryFull = 4, kPolyEveryCausal = 8;
constexpr int kFwdThreads = 384;   // 8 softmax warps + a 4-warp control group (MMA, producer, 2 idle)
constexpr int kKvStages = 4;
constexpr float kRescaleThreshold = 8.0f;   // in log2 units

struct FwdShared {
    uint64_t q_full[2], q_empty[2];
    uint64_t kv_full[kKvStages], kv_empty[kKvStages];
    uint64_t s_full[2], p_part[2][4], o_full[2], o_free[2];
    uint64_t work_full[2], work_empty[2];
    uint64_t stage_ready[2], stage_full[2];    // output staging buffer of a softmax group: free to write / written
    WorkItem work[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int D>
struct FwdCfg {
    static constexpr int kTileBytes = kTile * D * 2;   // one Q, K or V tile
    static constexpr int kBoxes = D / 64;               // TMA boxes per tile (64 columns = 128 bytes each)
    static constexpr int kBoxBytes = kTile * 128;
    static constexpr int kStageBytes = kTile * 128;     // 128 rows of 64 bf16 columns: what one TMA store box holds
    static constexpr int kOffStage = (2 + kKvStages) * kTileBytes;   // one staging buffer per softmax group
    static constexpr int kSmemBytes = kOffStage + 2 * kStageBytes + 1024;
    static constexpr uint32_t kS0 = 0, kS1 = 128, kO0 = 256, kO1 = 256 + D;   // tensor-memory columns
};

// Number of K/V tiles a Q tile starting at row r0 attends to (0 if the tile is past the end).
template <bool CAUSAL>
__device__ __forceinline__ int kv_tiles_for(int r0, int len) {
    if (r0 >= len) return 0;
    const int all = (len + kTile - 1) / kTile;
    if (!CAUSAL) return all;
    const int diag = r0 / kTile + 1;
    return diag < all ? diag : all;
}

template <int D>
__device__ __forceinline__ void load_tile(uint8_t* dst, const CUtensorMap* map, uint64_t* bar, int head, int row) {
    mbar_expect_tx(bar, FwdCfg<D>::kTileBytes);
#pragma unroll
    for (int b = 0; b < FwdCfg<D>::kBoxes; ++b)
        tma_load_3d(dst + b * FwdCfg<D>::kBoxBytes, map, bar, b * 64, head, row);
}

// The MMA warp runs its loop with all 32 lanes in lock step and only `leader` issues: every operand
// below is then warp-uniform, the descriptors are built once outside the loops, and a k-step costs
// one add per operand.  (tcgen05.mma issue blocks while the pipe is busy, and a lone thread executes
// dependent instructions several cycles apart, so each instruction between two MMAs is pipe idle time.)

// S = Q K^T for one 128x128 tile: both operands K-contiguous in shared memory.
// TRIM: the head dimension is smaller than the D columns the tiles hold (the rest are zeros), so only the
// first n_ks steps of 16 columns are multiplied; without it the loop is the full, compile-time one.
template <int D, bool TRIM>
__device__ __forceinline__ void issue_qk(uint32_t d_tmem, uint64_t q_desc, uint64_t k_desc, bool leader, int n_ks) {
    constexpr uint32_t idesc = make_idesc_bf16(128, 128, false, false);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        constexpr int kBox = FwdCfg<D>::kBoxBytes;
        const uint64_t off = (uint64_t)(((ks / 4) * kBox + (ks % 4) * 32) >> 4);
        if (leader && (!TRIM || ks < n_ks)) tc_mma_ss(d_tmem, q_desc + off, k_desc + off, idesc, ks > 0);
    }
}

// O (+)= P V: P from tensor memory (bf16 pairs per column), V with head_dim contiguous.
// `part` selects 32 of the tile's 128 keys: the product starts on the first part of P while the softmax
// group is still producing the rest, which shortens the chain S -> softmax -> PV -> next S.
// TRIM: only the first 16 * n_ks columns of O are computed (idesc_trim carries that width).
template <int D, bool TRIM>
__device__ __forceinline__ void issue_pv(uint32_t d_tmem, uint32_t p_tmem, uint64_t v_desc, bool accumulate, bool leader,
                                         int part, uint32_t idesc_trim) {
    const uint32_t idesc = TRIM ? idesc_trim : make_idesc_bf16(128, D, false, true);
#pragma unroll
    for (int k4 = 0; k4 < 2; ++k4) {
        const int ks = part * 2 + k4;
        if (leader) tc_mma_ts(d_tmem, p_tmem + ks * 8, v_desc + (uint64_t)((ks * 2048) >> 4), idesc, accumulate || ks > 0);
    }
}

// Softmax of a work item that is a single tile (a virtual sequence of at most 128 tokens, in which
// short sequences may have been merged): the row of a token sees only the positions of its own
// sequence, given by the per-token table.  Kept out of line so that the multi-tile loop of the common
// case is compiled exactly as it would be without this path.  Called by the 128 threads of softmax
// group 0 with the parities of their next s_full and o_full phases.
template <int D, bool CAUSAL>
__device__ __noinline__ void softmax_single_tile_item(FwdShared& sh, const FwdParams& p, const WorkItem w,
                                                      uint32_t s_tmem, uint32_t o_tmem, uint32_t s_parity,
                                                      uint32_t o_parity, const WaitGuard guard) {
    const int lane = threadIdx.x & 31;
    const int row = threadIdx.x & 127;
    const bool valid = row < w.len;
    int first_key = 0, end_key = w.len;
    if (valid) {
        const uint32_t b = p.bounds[(size_t)w.tok0 + row];
        first_key = (int)(b & 0xffu);
        end_key = (int)(b >> 8);
    }
    const int last_key = CAUSAL ? (row < end_key - 1 ? row : end_key - 1) : end_key - 1;
    mbar_wait(&sh.s_full[0], s_parity, guard);
    tc_fence_after();
    uint32_t s[128];
#pragma unroll
    for (int c = 0; c < 4; ++c) tmem_ld_x32(s_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 128; ++c)
        if (c > last_key || c < first_key) s[c] = 0xff800000u;         // -inf
    // this item is one dependent chain S -> softmax -> PV per CTA: eight maxima and two packed sums run
    // side by side instead of one 128-long chain each
    float part[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) part[c] = fmax3(__uint_as_float(s[c]), __uint_as_float(s[8 + c]), __uint_as_float(s[16 + c]));
#pragma unroll
    for (int c = 24; c < 120; c += 16) {
#pragma unroll
        for (int u = 0; u < 8; ++u) part[u] = fmax3(part[u], __uint_as_float(s[c + u]), __uint_as_float(s[c + 8 + u]));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) part[u] = fmaxf(part[u], __uint_as_float(s[120 + u]));
    const float m = fmaxf(fmax3(part[0], part[1], part[2]), fmax3(fmax3(part[3], part[4], part[5]), part[6], part[7]));
    const float neg_m = -m * p.scale_log2;
    const uint64_t sc2 = pack_f32x2(p.scale_log2, p.scale_log2), nm2 = pack_f32x2(neg_m, neg_m);
    uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float x0, x1;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[c * 32 + 2 * i]), __uint_as_float(s[c * 32 + 2 * i + 1])), sc2, nm2),
                         x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
            pk[i] = pack_bf16x2(p0, p1);
        }
        tmem_st_x16(s_tmem + c * 16, pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.p_part[0][c]);
    }
    float l;
    {
        float a0, a1, b0, b1;
        unpack_f32x2(sum2[0], a0, a1);
        unpack_f32x2(sum2[1], b0, b1);
        l = (a0 + a1) + (b0 + b1);
    }
    mbar_wait(&sh.o_full[0], o_parity, guard);
    tc_fence_after();
    const float inv_l = 1.0f / l;
    const size_t tok = (size_t)w.tok0 + (size_t)row;
    __nv_bfloat16* out = p.o + tok * p.row_stride + w.head * p.head_dim;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t acc[32];
        tmem_ld_x32(o_tmem + c * 32, acc);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
                uint4 val;
                val.x = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 0]) * inv_l, __uint_as_float(acc[v4 * 8 + 1]) * inv_l);
                val.y = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 2]) * inv_l, __uint_as_float(acc[v4 * 8 + 3]) * inv_l);
                val.z = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 4]) * inv_l, __uint_as_float(acc[v4 * 8 + 5]) * inv_l);
                val.w = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 6]) * inv_l, __uint_as_float(acc[v4 * 8 + 7]) * inv_l);
                if (c * 32 + v4 * 8 < p.head_dim) *reinterpret_cast<uint4*>(out + c * 32 + v4 * 8) = val;
            }
        }
    }
    if (valid) p.lse[(size_t)w.head * p.total_tokens + tok] = m * p.scale + __logf(l);
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.o_free[0]);
}

// Epilogue of a Q tile whose 128 rows all belong to the sequence: O = acc / l leaves tensor memory through a
// staging buffer in shared memory and TMA stores, 64 columns (one box) at a time.  A thread owns a row, so storing
// it directly costs 16 instructions of 32 scattered 16-byte pieces each, about a microsecond of the load/store
// unit per tile: as much as a key tile's softmax, which is what short work items cannot afford (uniform batches
// of 256-token sequences: forward 0.41 -> 0.36 ms).  Kept out of line so that the loop over key tiles is compiled
// exactly as it would be without it (inlined it cost the long-sequence forward 6 %).  Called by the 128 threads
// of a softmax group; n_staged = boxes this group has stored so far (the parity of its two barriers).
template <int D>
__device__ __noinline__ void store_whole_tile(FwdShared& sh, const CUtensorMap* tmap_o, uint8_t* stage, uint32_t o_tmem,
                                              float inv_l, int t, int head, int tok_row0, uint32_t n_staged,
                                              const WaitGuard guard) {
    const int lane = threadIdx.x & 31, row_in_tile = threadIdx.x & 127;
    const bool issuer = row_in_tile == 0;
#pragma unroll
    for (int half = 0; half < D / 64; ++half, ++n_staged) {
        uint32_t acc[64];
        tmem_ld_x32(o_tmem + half * 64, *reinterpret_cast<uint32_t(*)[32]>(&acc[0]));
        tmem_ld_x32(o_tmem + half * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[32]));
        tmem_wait_ld();
        if (half == D / 64 - 1) {       // O has left tensor memory: the next item's P V may start
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.o_free[t]);
        }
        if (issuer) {
            bulk_store_wait_read();              // the previous store has read the staging buffer
            mbar_arrive(&sh.stage_ready[t]);
        }
        mbar_wait(&sh.stage_ready[t], n_staged & 1u, guard);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint4 val;
            val.x = pack_bf16x2(__uint_as_float(acc[c * 8 + 0]) * inv_l, __uint_as_float(acc[c * 8 + 1]) * inv_l);
            val.y = pack_bf16x2(__uint_as_float(acc[c * 8 + 2]) * inv_l, __uint_as_float(acc[c * 8 + 3]) * inv_l);
            val.z = pack_bf16x2(__uint_as_float(acc[c * 8 + 4]) * inv_l, __uint_as_float(acc[c * 8 + 5]) * inv_l);
            val.w = pack_bf16x2(__uint_as_float(acc[c * 8 + 6]) * inv_l, __uint_as_float(acc[c * 8 + 7]) * inv_l);
            *reinterpret_cast<uint4*>(stage + sw128_offset((uint32_t)row_in_tile, (uint32_t)c)) = val;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.stage_full[t]);
        if (issuer) {
            if (mbar_wait(&sh.stage_full[t], n_staged & 1u, guard)) tma_store_3d(tmap_o, stage, half * 64, head, tok_row0);
            bulk_store_commit();
        }
    }
}

// EARLY_Q: release a Q tile's slot as soon as its last S product has been issued (see the MMA warp).
// TRIM: head_dim is at most D - 16, so the products skip the zero-padded columns: S sums over
// ceil(head_dim / 16) steps instead of D / 16 and O is 16 * ceil(head_dim / 16) columns wide (head_dim 72,
// the width of the paper's second model, does 5/8 of the padded work).
template <int D, bool CAUSAL, bool EARLY_Q, bool TRIM>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                const __grid_constant__ FwdParams p) {
    using Cfg = FwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sKV = smem + 2 * Cfg::kTileBytes;
    __shared__ FwdShared sh;

    const int tid = threadIdx.x;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);     // via a shuffle: provably uniform within the warp
    const int lane = tid & 31;
    const WaitGuard guard{&sh.abort_flag, &p.sched.hdr->status};

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.q_full[i], 1);
            mbar_init(&sh.q_empty[i], 1);
            mbar_init(&sh.s_full[i], 1);
            for (int k = 0; k < 4; ++k) mbar_init(&sh.p_part[i][k], 4);   // one arrival per softmax warp per 32 keys of P
            mbar_init(&sh.o_full[i], 1);
            mbar_init(&sh.o_free[i], 4);
            mbar_init(&sh.work_full[i], 1);
            mbar_init(&sh.work_empty[i], 9);   // 8 softmax warps + the MMA thread
            mbar_init(&sh.stage_ready[i], 1);
            mbar_init(&sh.stage_full[i], 4);   // one arrival per warp of the group
        }
        for (int i = 0; i < kKvStages; ++i) {
            mbar_init(&sh.kv_full[i], 1);
            mbar_init(&sh.kv_empty[i], 1);
        }
        sh.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(&sh.tmem_base, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // when this CTA started and (at the end) when it ran out of work: the spread over CTAs measures the balance
    if (tid == 0 && blockIdx.x < kMaxCtas) {
        p.sched.spans[0 * kMaxCtas + blockIdx.x].begin_ns = global_timer_ns();
        if (blockIdx.x == 0) p.sched.hdr->n_ctas[0] = gridDim.x < kMaxCtas ? gridDim.x : kMaxCtas;
    }

    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    if (warp == 9) {
        // ---------------------------------------------------------------- scheduler + TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmap_q);
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            const uint32_t n_items = p.sched.hdr->n_items;
            uint32_t n_work = 0, kv_count = 0, q_use[2] = {0, 0};
            while (true) {
                const uint32_t slot = n_work & 1u;
                if (n_work >= 2) mbar_wait(&sh.work_empty[slot], ((n_work >> 1) - 1) & 1u, guard);
                const uint32_t item = atomicAdd(&p.sched.hdr->work_counter, 1u);
                WorkItem w;
                if (item < n_items && !sh.abort_flag) {
                    w = decode_item(p.sched, p.cu_seqlens, item, kFwdRowsPerItem, p.n_heads, CAUSAL);
                } else {
                    w.tok0 = 0; w.len = -1; w.head = 0; w.blk = 0; w.tile0 = 0;
                }
                sh.work[slot] = w;
                mbar_arrive(&sh.work_full[slot]);
                ++n_work;
                if (w.len < 0) break;

                const int r0 = w.blk * kFwdRowsPerItem;
                const int nkv_t[2] = {kv_tiles_for<CAUSAL>(r0, w.len), kv_tiles_for<CAUSAL>(r0 + kTile, w.len)};
                const int nkv = nkv_t[0] > nkv_t[1] ? nkv_t[0] : nkv_t[1];
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (nkv_t[t] == 0) continue;
                    if (q_use[t] >= 1) mbar_wait(&sh.q_empty[t], (q_use[t] - 1) & 1u, guard);
                    load_tile<D>(sQ + t * Cfg::kTileBytes, &tmap_q, &sh.q_full[t], w.head, w.tok0 + r0 + t * kTile);
                    ++q_use[t];
                }
                for (int j = 0; j < nkv; ++j) {
#pragma unroll
                    for (int which = 0; which < 2; ++which) {
                        const uint32_t stage = kv_count % kKvStages, fill = kv_count / kKvStages;
                        if (fill >= 1) mbar_wait(&sh.kv_empty[stage], (fill - 1) & 1u, guard);
                        load_tile<D>(sKV + stage * Cfg::kTileBytes, which == 0 ? &tmap_k : &tmap_v, &sh.kv_full[stage],
                                     w.head, w.tok0 + j * kTile);
                        ++kv_count;
                    }
                }
            }
        }
    } else if (warp == 8) {
        // ---------------------------------------------------------------- MMA issue
        {
            const bool leader = elect_one();
            uint32_t n_work = 0, kv_base = 0, use[2] = {0, 0}, n_p[2] = {0, 0};
            const uint64_t q_desc[2] = {make_sdesc_sw128(smem_u32(sQ), 16, 1024),
                                        make_sdesc_sw128(smem_u32(sQ) + Cfg::kTileBytes, 16, 1024)};
            const uint64_t kv_km0 = make_sdesc_sw128(smem_u32(sKV), 16, 1024);                 // K: head_dim contiguous
            const uint64_t kv_mn0 = make_sdesc_sw128(smem_u32(sKV), Cfg::kBoxBytes, 1024);     // V: head_dim contiguous = N
            constexpr uint32_t kStageStep = Cfg::kTileBytes >> 4;
            const uint32_t s_tmem[2] = {tmem + Cfg::kS0, tmem + Cfg::kS1};
            const uint32_t o_tmem[2] = {tmem + Cfg::kO0, tmem + Cfg::kO1};
            const int n_ks = TRIM ? (p.head_dim + 15) >> 4 : D / 16;
            const uint32_t idesc_pv = make_idesc_bf16(128, n_ks * 16, false, true);
            auto kv_wait = [&](uint32_t idx) {
                mbar_wait(&sh.kv_full[idx % kKvStages], (idx / kKvStages) & 1u, guard);
            };
            auto commit = [&](uint64_t* bar) { if (leader) tc_commit(bar); };
            while (true) {
                const uint32_t slot = n_work & 1u;
                const bool got = mbar_wait(&sh.work_full[slot], (n_work >> 1) & 1u, guard);
                if (!__all_sync(0xffffffffu, got)) break;
                const WorkItem w = sh.work[slot];
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.work_empty[slot]);
                ++n_work;
                if (w.len < 0) break;
                const int r0 = w.blk * kFwdRowsPerItem;
                const int nkv_t[2] = {kv_tiles_for<CAUSAL>(r0, w.len), kv_tiles_for<CAUSAL>(r0 + kTile, w.len)};
                const int nkv = nkv_t[0] > nkv_t[1] ? nkv_t[0] : nkv_t[1];

                // S_t(0) for both tiles
                kv_wait(kv_base);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (nkv_t[t] == 0) continue;
                    mbar_wait(&sh.q_full[t], use[t] & 1u, guard);
                    tc_fence_after();
                    issue_qk<D, TRIM>(s_tmem[t], q_desc[t], kv_km0 + (kv_base % kKvStages) * kStageStep, leader, n_ks);
                    commit(&sh.s_full[t]);
                    // When items are short (a query block sees a few key tiles: causal masks, batches of short
                    // sequences) a Q tile is released as soon as its last S product is issued, so that the next
                    // item's Q load runs while this item's last PV products do instead of after them (config 2
                    // forward 1.05 -> 1.01 ms, spatial axis of the 2-D workload 1.97 -> 1.84 ms).  On long items the
                    // two extra tests per key step cost the MMA warp more than the early load gains (config 3
                    // forward 16.4 -> 16.9 ms), so the host picks the variant by mask and longest sequence.
                    if (EARLY_Q && nkv_t[t] == 1) commit(&sh.q_empty[t]);
                }
                commit(&sh.kv_empty[kv_base % kKvStages]);

                for (int j = 0; j < nkv; ++j) {
                    const uint32_t iv = kv_base + 2 * j + 1, ik = kv_base + 2 * j + 2;
                    const uint32_t st_v = iv % kKvStages, st_k = ik % kKvStages;
                    const bool has_next = j + 1 < nkv;
                    kv_wait(iv);
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (t == 1 && has_next) kv_wait(ik);
                        if (t == 1 && j + 1 < nkv_t[0]) {      // S_0(j+1) goes between the two PV products
                            tc_fence_after();
                            issue_qk<D, TRIM>(s_tmem[0], q_desc[0], kv_km0 + st_k * kStageStep, leader, n_ks);
                            commit(&sh.s_full[0]);
                            if (EARLY_Q && j + 2 == nkv_t[0]) commit(&sh.q_empty[0]);
                        }
                        if (j < nkv_t[t]) {
                            if (j == 0 && use[t] >= 1) mbar_wait(&sh.o_free[t], (use[t] - 1) & 1u, guard);
#pragma unroll
                            for (int part = 0; part < 4; ++part) {
                                mbar_wait(&sh.p_part[t][part], n_p[t] & 1u, guard);
                                tc_fence_after();
                                issue_pv<D, TRIM>(o_tmem[t], s_tmem[t], kv_mn0 + st_v * kStageStep, j > 0, leader, part, idesc_pv);
                            }
                            ++n_p[t];
                            if (j == nkv_t[t] - 1) commit(&sh.o_full[t]);
                        }
                    }
                    commit(&sh.kv_empty[st_v]);
                    if (j + 1 < nkv_t[1]) {
                        issue_qk<D, TRIM>(s_tmem[1], q_desc[1], kv_km0 + st_k * kStageStep, leader, n_ks);
                        commit(&sh.s_full[1]);
                        if (EARLY_Q && j + 2 == nkv_t[1]) commit(&sh.q_empty[1]);
                    }
                    if (has_next) commit(&sh.kv_empty[st_k]);
                }
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (nkv_t[t] == 0) continue;
                    if (!EARLY_Q) commit(&sh.q_empty[t]);
                    ++use[t];
                }
                kv_base += 2 * nkv;
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        // ---------------------------------------------------------------- softmax groups
        const int t = warp >> 2;                        // Q tile of this group
        const int row_in_tile = tid & 127;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_tmem = tmem + lane_base + (t == 0 ? Cfg::kS0 : Cfg::kS1);
        const uint32_t o_tmem = tmem + lane_base + (t == 0 ? Cfg::kO0 : Cfg::kO1);
        uint32_t n_work = 0, n_s = 0, use = 0, n_staged = 0;
        while (true) {
            const uint32_t slot = n_work & 1u;
            const bool got = mbar_wait(&sh.work_full[slot], (n_work >> 1) & 1u, guard);
            if (!__all_sync(0xffffffffu, got)) break;
            const WorkItem w = sh.work[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.work_empty[slot]);
            ++n_work;
            if (w.len < 0) break;
            if (p.bounds != nullptr && w.len <= kTile) {      // one tile, possibly several merged sequences
                if (t == 0) {
                    softmax_single_tile_item<D, CAUSAL>(sh, p, w, s_tmem, o_tmem, n_s & 1u, use & 1u, guard);
                    ++n_s;
                    ++use;
                }
                continue;
            }
            const int r_tile = w.blk * kFwdRowsPerItem + t * kTile;
            const int nkv = kv_tiles_for<CAUSAL>(r_tile, w.len);
            if (nkv == 0) continue;
            const int row = r_tile + row_in_tile;       // row inside the sequence (may be >= len)

            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < nkv; ++j) {
                mbar_wait(&sh.s_full[t], n_s & 1u, guard);
                ++n_s;
                tc_fence_after();
                uint32_t s[128];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld_x32(s_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                tmem_wait_ld();

                const bool boundary = (j == nkv - 1) && (CAUSAL || (w.len & (kTile - 1)) != 0);
                if (boundary) {
                    const int last_key = CAUSAL ? (row < w.len - 1 ? row : w.len - 1) : w.len - 1;
                    const int n_valid = last_key - j * kTile + 1;     // >= 1
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= n_valid) s[c] = 0xff800000u;         // -inf
                }
                float part[8];      // eight independent chains instead of one 128-long one, three-input maxima
#pragma unroll
                for (int c = 0; c < 8; ++c) part[c] = fmax3(__uint_as_float(s[c]), __uint_as_float(s[8 + c]), __uint_as_float(s[16 + c]));
#pragma unroll
                for (int c = 24; c < 120; c += 16) {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        part[u] = fmax3(part[u], __uint_as_float(s[c + u]), __uint_as_float(s[c + 8 + u]));
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) part[u] = fmaxf(part[u], __uint_as_float(s[120 + u]));
                const float mx = fmaxf(fmax3(part[0], part[1], part[2]), fmax3(fmax3(part[3], part[4], part[5]), part[6], part[7]));

                const bool need = (mx - m) * p.scale_log2 > kRescaleThreshold;
                if (__any_sync(0xffffffffu, need)) {
                    // the branch is warp-wide (the accumulator rescale below is a warp-collective tensor-memory
                    // access), but each row raises its own maximum only if it needs to itself: what a row
                    // computes must not depend on the other rows of its warp, some of which may belong to the
                    // next sequence of the packed batch
                    const float m_new = need ? fmaxf(m, mx) : m;
                    const float factor = need ? fast_exp2((m - m_new) * p.scale_log2) : 1.0f;
                    m = m_new;
                    l *= factor;
                    if (j > 0) {
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t acc[32];
                            tmem_ld_x32(o_tmem + c * 32, acc);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * factor);
                            tmem_st_x32(o_tmem + c * 32, acc);
                        }
                    }
                }
                const float neg_m = -m * p.scale_log2;
                const uint64_t sc2 = pack_f32x2(p.scale_log2, p.scale_log2), nm2 = pack_f32x2(neg_m, neg_m);
                uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        // scaled, shifted scores of two keys in one packed FMA; one pair in kPolyEvery takes
                        // its exponentials from the FMA pipe, the others from the special-function unit,
                        // which a 128 x 128 tile would otherwise keep busy as long as its two MMAs take
                        const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[c * 32 + 2 * i]),
                                                                 __uint_as_float(s[c * 32 + 2 * i + 1])), sc2, nm2);
                        float p0, p1;
                        constexpr int kPolyEvery = CAUSAL ? kPolyEveryCausal : kPolyEveryFull;
                        if (kPolyEvery > 0 && (i % (kPolyEvery > 0 ? kPolyEvery : 1)) == kPolyEvery - 1) {
                            poly_exp2_pair(x2, p0, p1);
                        } else {
                            float x0, x1;
                            unpack_f32x2(x2, x0, x1);
                            p0 = fast_exp2(x0);
                            p1 = fast_exp2(x1);
                        }
                        sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
                        pk[i] = pack_bf16x2(p0, p1);
                    }
                    tmem_st_x16(s_tmem + c * 16, pk);
                    // these 32 keys of P are in tensor memory: the PV product may use them
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.p_part[t][c]);
                }
                {
                    float a0, a1, b0, b1;
                    unpack_f32x2(sum2[0], a0, a1);
                    unpack_f32x2(sum2[1], b0, b1);
                    l += (a0 + a1) + (b0 + b1);
                }
            }

            // epilogue: O = acc / l, lse = m*scale + ln l
            mbar_wait(&sh.o_full[t], use & 1u, guard);
            ++use;
            tc_fence_after();
            const float inv_l = 1.0f / l;
            const bool valid = row < w.len;
            const size_t tok = (size_t)w.tok0 + (size_t)row;
            if (r_tile + kTile <= w.len) {
                // every row of the tile belongs to the sequence: it leaves through shared memory and TMA stores
                store_whole_tile<D>(sh, &tmap_o, smem + Cfg::kOffStage + t * Cfg::kStageBytes, o_tmem, inv_l, t, w.head,
                                    w.tok0 + r_tile, n_staged, guard);
                n_staged += D / 64;
                p.lse[(size_t)w.head * p.total_tokens + tok] = m * p.scale + __logf(l);
                continue;
            }
            __nv_bfloat16* out = p.o + tok * p.row_stride + w.head * p.head_dim;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t acc[32];
                tmem_ld_x32(o_tmem + c * 32, acc);
                tmem_wait_ld();
                if (valid) {
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4 val;
                        val.x = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 0]) * inv_l, __uint_as_float(acc[v4 * 8 + 1]) * inv_l);
                        val.y = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 2]) * inv_l, __uint_as_float(acc[v4 * 8 + 3]) * inv_l);
                        val.z = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 4]) * inv_l, __uint_as_float(acc[v4 * 8 + 5]) * inv_l);
                        val.w = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 6]) * inv_l, __uint_as_float(acc[v4 * 8 + 7]) * inv_l);
                        if (c * 32 + v4 * 8 < p.head_dim) *reinterpret_cast<uint4*>(out + c * 32 + v4 * 8) = val;
                    }
                }
            }
            if (valid) p.lse[(size_t)w.head * p.total_tokens + tok] = m * p.scale + __logf(l);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.o_free[t]);
        }
        if ((tid & 127) == 0) bulk_store_wait_all();     // this group's stores are complete before the CTA ends
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && blockIdx.x < kMaxCtas) p.sched.spans[0 * kMaxCtas + blockIdx.x].end_ns = global_timer_ns();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int D, bool CAUSAL, bool EARLY_Q, bool TRIM>
static cudaError_t launch_one(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                              const FwdParams& p, int n_ctas, cudaStream_t stream) {
    auto kern = attn_fwd_kernel<D, CAUSAL, EARLY_Q, TRIM>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<D>::kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<n_ctas, kFwdThreads, FwdCfg<D>::kSmemBytes, stream>>>(tq, tk, tv, to, p);
    return cudaGetLastError();
}

template <int D, bool TRIM>
static cudaError_t launch_masked(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                                 const FwdParams& p, bool causal, bool short_items, int n_ctas, cudaStream_t stream) {
    if (causal) return launch_one<D, true, true, TRIM>(tq, tk, tv, to, p, n_ctas, stream);
    return short_items ? launch_one<D, false, true, TRIM>(tq, tk, tv, to, p, n_ctas, stream)
                       : launch_one<D, false, false, TRIM>(tq, tk, tv, to, p, n_ctas, stream);
}

cudaError_t launch_attn_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                            const FwdParams& p, int head_dim, bool causal, bool short_items, int n_ctas, cudaStream_t stream) {
    if (head_dim > 112) return launch_masked<128, false>(tq, tk, tv, to, p, causal, short_items, n_ctas, stream);
    if (head_dim > 64) return launch_masked<128, true>(tq, tk, tv, to, p, causal, short_items, n_ctas, stream);
    return launch_masked<64, false>(tq, tk, tv, to, p, causal, short_items, n_ctas, stream);
}

}  // namespace dcp
