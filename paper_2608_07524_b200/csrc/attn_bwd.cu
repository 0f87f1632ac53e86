// Backward packed variable-length attention for sm_100a (main kernel).
//
// One persistent CTA per SM.  A work item is (sequence, head, 128 keys); the CTA keeps that K and V
// tile in shared memory and walks over every Q tile that sees it.  Everything is computed in the
// transposed orientation, keys on tensor-memory lanes and queries on columns, so that P^T can feed
// the dV product straight from tensor memory:
//
//     S'^T  = K Q^T - 1 (lse/scale)^T   (tcgen05, fp32 in tensor memory)
//     P^T   = exp2(S'^T * scale*log2e), masked                     -> bf16, overwrites S'^T
//     dP'^T = V dO^T - 1 D^T
//     dS^T  = P^T o dP'^T                                          -> bf16, shared memory
//     dV  += P^T dO          dK += dS^T Q          dQ_tile = dS K  (dQ aliases dP^T's columns)
//
// The per-query terms -lse/scale and -D are columns in this orientation; instead of every thread
// reading them (a shared-memory broadcast costs one wavefront per value, on the port that feeds the
// MMAs), they are added by one extra K=16 MMA per product: A = a constant tile of ones, B = a
// [128 queries x 16] bf16 tile holding each term split into three bf16 parts (24 bits, exact sum in
// the fp32 accumulator), prepared per (tile, head) by the pre kernel and fetched by bulk copy.
//
// dQ tiles are added into an fp32 accumulator in global memory with vector atomics because every
// key block of a sequence contributes to the same query rows.  The accumulator is a workspace, so
// its layout is chosen for the atomics: per (tile, head) a block [d/4][128 rows][4 floats], which
// makes the 32 rows a warp holds contiguous (full 32-byte sectors, four 128-byte lines per
// instruction instead of 32 scattered ones); a small kernel converts it to [T, H, d] bf16 later.
// These 64 KB per (Q tile, K tile) pair are what bounds the kernel: the SM's path to L2 moves about
// 15-25 bytes per clock for reductions, per-thread atomics and shared-memory bulk reductions alike,
// and the atomics share the load/store unit with the compute warps' dS^T stores; with the atomics
// compiled out the same kernel runs a third faster.  What helps is pausing the drain warps briefly
// between groups of atomics (see kRedGroup).  Measured and rejected: pacing by spinning on the clock
// (the spin takes issue slots from the compute warps), bulk reductions from a 16 KB staging buffer,
// atomics into an L2-hot block (same time, so the limit is on the SM's side), dK before dQ, and
// staggering the Q walk of neighbouring key blocks.
// dK and dV stay in tensor memory for the whole item and are written once (dK scaled by the
// softmax scale).
//
// The MMA warp runs its loop warp-uniformly and an elected lane issues: a tcgen05.mma issue blocks,
// and a lone diverged thread that also computes descriptors pays 80-100 cycles per instruction, so
// descriptors are built once per item and a k-step is a constant add.  P^T is published in two
// parts (the first 32 query columns of each column group first), so the dV product starts on
// those while the rest is still being exponentiated.
//
// Roles:  warps 0-7 compute (two groups, each owns 64 of the 128 query columns, one key per thread),
//         warp 8 MMA issue, warp 9 scheduler + TMA producer + per-row statistics staging
//         (warps 10-11 idle: the control group of four gives most of its registers away),
//         warps 12-15 dQ drain (tensor memory -> global atomics).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sched.cuh"
#include "sm100_ptx.cuh"

namespace dcp {

// The drain warps pause after every kRedGroup vector atomics, and warp k of the four starts k pauses
// late.  Issued back to back, a tile's 64 KB of atomics fill the SM's queue towards L2, and the TMA
// requests and shared-memory stores of the other warps wait behind them; short sleeps (which, unlike
// a spin on the clock, take no issue slots) let those through.  __nanosleep rounds down to steps of
// about 128 ns here (100 ns had no effect, 150-250 ns the same effect), so the values sit in the
// middle of a step.  Backward main kernel alone on config 3: 60.2 ms without any pause, 58.3 with the
// pauses, 55.8 with the stagger as well; two steps per pause or per stagger, or a pause after every
// second atomic, cost 57-85 ms.  In the power-capped bench loop: 61.7 -> 58.1 ms.
constexpr int kRedGroup = 4;
constexpr unsigned kRedSleepNs = 192;        // one step
constexpr unsigned kRedStaggerNs = 128;      // per drain warp, plus half a step
constexpr int kBwdThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct BwdCfg {
    static constexpr int kTileBytes = kTile * D * 2;     // K, V, Q or dO tile
    static constexpr int kBoxBytes = kTile * 128;
    static constexpr int kBoxes = D / 64;
    static constexpr int kDsBytes = kTile * kTile * 2;   // dS^T tile, bf16
    // shared-memory map (offsets from a 1024-byte aligned base)
    static constexpr int kOffK = 0;
    static constexpr int kOffV = kTileBytes;
    static constexpr int kQStages = 2;                     // Q is needed early (S^T) and late (dK)
    static constexpr int kOffQ = 2 * kTileBytes;
    static constexpr int kOffDo = (2 + kQStages) * kTileBytes;          // dO lives only from dP^T to dV: one stage
    static constexpr int kOffDs = (3 + kQStages) * kTileBytes;
    static constexpr int kStatBytes = kTile * 16 * 2;      // [128 x 16] bf16 tile, K-contiguous, no swizzle
    static constexpr int kOffOnes = kOffDs + kDsBytes;     // two constant tiles: ones in columns 0-2 / 8-10
    static constexpr int kOffStat = kOffOnes + 2 * kStatBytes;   // 2 slots of per-query terms
    static constexpr int kOffCtl = kOffStat + 2 * kStatBytes;
    static constexpr int kSmemBytes = kOffCtl + 320;
    static_assert(kSmemBytes <= 232448, "exceeds the 227 KB a CTA may use");
    // tensor-memory columns
    static constexpr uint32_t kSt = 0, kDp = 128, kDv = 256, kDk = 384;
};

struct BwdControl {
    uint64_t work_full[2], work_empty[2];
    uint64_t kv_full, kv_empty;
    uint64_t q_full[2], q_empty[2], do_full, do_empty, stat_full[2], stat_empty[2];
    uint64_t s_full, p_half, p_full, dp_full, ds_full, ds_free, dq_full, dq_free, dkv_full, dkv_free;
    uint64_t stage_ready[2], stage_full[2];   // dK / dV staging (the dS^T buffer at the end of an item), per column half
    WorkItem work[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};
static_assert(sizeof(BwdControl) <= 320, "control block must fit its slot");

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int D>
__device__ __forceinline__ void bwd_load_tile(uint8_t* dst, const CUtensorMap* map, uint64_t* bar, int head, int row) {
#pragma unroll
    for (int b = 0; b < BwdCfg<D>::kBoxes; ++b)
        tma_load_3d(dst + b * BwdCfg<D>::kBoxBytes, map, bar, b * 64, head, row);
}

// Compute-warp work of an item that is a single tile pair (a virtual sequence of at most 128 tokens,
// in which short sequences may have been merged): P^T and dS^T with a key seen only by the queries at
// the positions of its own sequence, which the per-token table gives.  Kept out of line so that the
// loop of the common case is compiled exactly as it would be without this path.  `g` is the running
// tile-pair count of the calling thread (it selects the barrier phases).
template <bool CAUSAL>
__device__ __noinline__ void compute_single_tile_item(BwdControl& sh, const BwdParams& p, const WorkItem w, uint32_t st_tmem,
                                                      uint32_t dp_tmem, uint8_t* ds_row, int half, int key_in_tile,
                                                      uint32_t g, const WaitGuard guard) {
    const int lane = threadIdx.x & 31;
    const bool key_valid = key_in_tile < w.len;
    int q_lo = 0, q_hi = 0;
    if (key_valid) {
        const uint32_t b = p.bounds[(size_t)w.tok0 + key_in_tile];
        q_lo = (int)(b & 0xffu);
        q_hi = (int)(b >> 8);
    }
    if (CAUSAL && key_in_tile > q_lo) q_lo = key_in_tile;     // a key is seen from its own position on
    float pf[64];
    mbar_wait(&sh.s_full, g & 1u, guard);
    tc_fence_after();
    {
        uint32_t sr[64];
        tmem_ld_x32(st_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
        tmem_ld_x32(st_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int q_first = half * 64 + c * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const int qi = q_first + e;
                const float x = fast_exp2(__uint_as_float(sr[c * 32 + e]) * p.scale_log2);
                pf[c * 32 + e] = (qi >= q_lo && qi < q_hi) ? x : 0.f;
            }
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = pack_bf16x2(pf[c * 32 + 2 * e], pf[c * 32 + 2 * e + 1]);
            tmem_st_x16(st_tmem + c * 16, pk);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(c == 0 ? &sh.p_half : &sh.p_full);
        }
    }
    mbar_wait(&sh.dp_full, g & 1u, guard);
    if (g >= 1) mbar_wait(&sh.ds_free, (g - 1) & 1u, guard);
    tc_fence_after();
    {
        uint32_t dr[64];
        tmem_ld_x32(dp_tmem, *reinterpret_cast<uint32_t(*)[32]>(&dr[0]));
        tmem_ld_x32(dp_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&dr[32]));
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                pk[e] = pack_bf16x2(pf[c * 8 + 2 * e] * __uint_as_float(dr[c * 8 + 2 * e]),
                                    pf[c * 8 + 2 * e + 1] * __uint_as_float(dr[c * 8 + 2 * e + 1]));
            *reinterpret_cast<uint4*>(ds_row + sw128_offset(key_in_tile, c)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    }
    fence_async_smem();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.ds_full);
}

// Item epilogue for a key block whose 128 rows all belong to the sequence (head_dim > 64): dV, then dK, leave
// tensor memory through shared memory and TMA stores.  A thread owns a key row, so storing it directly sends 16-byte
// pieces of 32 different rows per instruction: 4096 requests per item through the SM's outbound port, which the dQ
// reductions already keep busy (without these stores the main kernel is 7 % faster on config 2 and the spatial
// axis, measured).  The staging area is the dS^T buffer, idle between the last product of an item and the first
// dS^T of the next: each group of four warps (one 64-column half = one TMA box) fills its 16 KB, its first thread
// stores the box and the group waits until the store has read the buffer.  Out of line, so that the per-tile loop
// of the compute warps is compiled as it would be without it.  n_staged = boxes this group has staged so far.
template <int D>
__device__ __noinline__ void store_dkv_staged(BwdControl& sh, const CUtensorMap* tmap_dk, const CUtensorMap* tmap_dv, uint8_t* stage,
                                              uint32_t tmem_row, int half, int head, int tok_row0, float scale, uint32_t n_staged,
                                              const WaitGuard guard) {
    using Cfg = BwdCfg<D>;
    const int lane = threadIdx.x & 31, key_in_tile = threadIdx.x & 127;
    const bool issuer = key_in_tile == 0;
#pragma unroll
    for (int which = 0; which < 2; ++which, ++n_staged) {
        const uint32_t src = tmem_row + (which == 0 ? Cfg::kDv : Cfg::kDk) + half * 64;
        const float mul = which == 0 ? 1.0f : scale;
        uint32_t acc[64];
        tmem_ld_x32(src, *reinterpret_cast<uint32_t(*)[32]>(&acc[0]));
        tmem_ld_x32(src + 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[32]));
        tmem_wait_ld();
        if (which == 1) {               // dV and dK have left tensor memory: the next item may accumulate
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.dkv_free);
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint4 val;
            val.x = pack_bf16x2(__uint_as_float(acc[c * 8 + 0]) * mul, __uint_as_float(acc[c * 8 + 1]) * mul);
            val.y = pack_bf16x2(__uint_as_float(acc[c * 8 + 2]) * mul, __uint_as_float(acc[c * 8 + 3]) * mul);
            val.z = pack_bf16x2(__uint_as_float(acc[c * 8 + 4]) * mul, __uint_as_float(acc[c * 8 + 5]) * mul);
            val.w = pack_bf16x2(__uint_as_float(acc[c * 8 + 6]) * mul, __uint_as_float(acc[c * 8 + 7]) * mul);
            *reinterpret_cast<uint4*>(stage + sw128_offset((uint32_t)key_in_tile, (uint32_t)c)) = val;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.stage_full[half]);
        if (issuer) {
            if (mbar_wait(&sh.stage_full[half], n_staged & 1u, guard))
                tma_store_3d(which == 0 ? tmap_dv : tmap_dk, stage, half * 64, head, tok_row0);
            bulk_store_commit();
            bulk_store_wait_read();      // the store has read the buffer: dK, or the next item's dS^T, may overwrite it
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.stage_ready[half]);
        mbar_wait(&sh.stage_ready[half], n_staged & 1u, guard);
    }
}

// TRIM: head_dim is at most D - 16, so the products skip the zero-padded columns: S^T and dP^T sum over
// ceil(head_dim / 16) steps instead of D / 16; dV, dK and dQ are 16 * ceil(head_dim / 16) columns wide, and so
// is what the drain warps add to the accumulator.
template <int D, bool CAUSAL, bool TRIM>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_do,
                const __grid_constant__ CUtensorMap tmap_dk, const __grid_constant__ CUtensorMap tmap_dv,
                const __grid_constant__ BwdParams p) {
    using Cfg = BwdCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    BwdControl& sh = *reinterpret_cast<BwdControl*>(smem + Cfg::kOffCtl);

    const int tid = threadIdx.x;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);     // via a shuffle: provably uniform within the warp
    const int lane = tid & 31;
    const WaitGuard guard{&sh.abort_flag, &p.sched.hdr->status};

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.work_full[i], 1);
            mbar_init(&sh.work_empty[i], 13);   // 8 compute warps + 4 drain warps + the MMA thread
            mbar_init(&sh.stat_full[i], 1);
            mbar_init(&sh.stat_empty[i], 1);
        }
        for (int i = 0; i < Cfg::kQStages; ++i) {
            mbar_init(&sh.q_full[i], 1);
            mbar_init(&sh.q_empty[i], 1);
        }
        mbar_init(&sh.do_full, 1);
        mbar_init(&sh.do_empty, 1);
        mbar_init(&sh.kv_full, 1);
        mbar_init(&sh.kv_empty, 1);
        mbar_init(&sh.s_full, 1);
        mbar_init(&sh.p_half, 8);     // first 32 query columns of each group's P^T written
        mbar_init(&sh.p_full, 8);
        mbar_init(&sh.dp_full, 1);
        mbar_init(&sh.ds_full, 8);
        mbar_init(&sh.ds_free, 1);
        mbar_init(&sh.dq_full, 1);
        mbar_init(&sh.dq_free, 4);
        mbar_init(&sh.dkv_full, 1);
        mbar_init(&sh.dkv_free, 8);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.stage_ready[i], 4);   // one arrival per warp of the half
            mbar_init(&sh.stage_full[i], 4);
        }
        sh.abort_flag = 0;
        fence_mbar_init();
        // the swizzled tile layout needs a 1024-byte aligned base; refuse to run otherwise
        if ((smem_u32(smem) & 1023u) != 0) {
            sh.abort_flag = 1;
            atomicMax(&p.sched.hdr->status, (uint32_t)kStatusBadSmemAlign);
        }
    }
    if (warp == 0) {
        tmem_alloc(&sh.tmem_base, 512);
        tmem_relinquish();
    }
    {   // constant A operands of the rank-1 MMAs: [128 keys x 16] with ones in columns 0-2 (adds the lse
        // term to S^T) and in columns 8-10 (adds the D term to dP^T).  Layout: 8x8 core matrices of
        // 128 bytes, row groups 128 bytes apart, the two column halves 2048 bytes apart.
        uint32_t* ones = reinterpret_cast<uint32_t*>(smem + Cfg::kOffOnes);
        for (int i = tid; i < 2 * Cfg::kStatBytes / 4; i += kBwdThreads) {
            const int tile = i / (Cfg::kStatBytes / 4), w32 = i % (Cfg::kStatBytes / 4);
            const int half = w32 / 512, in_row = w32 % 4;            // 32-bit word inside a 16-byte row chunk
            const bool on = half == tile;                            // tile 0: first column half, tile 1: second
            ones[i] = !on ? 0u : in_row == 0 ? 0x3f803f80u : in_row == 1 ? 0x00003f80u : 0u;   // 1,1 | 1,0 | 0..
        }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // when this CTA started and (at the end) when it ran out of work: the spread over CTAs measures the balance
    if (tid == 0 && blockIdx.x < kMaxCtas) {
        p.sched.spans[1 * kMaxCtas + blockIdx.x].begin_ns = global_timer_ns();
        if (blockIdx.x == 0) p.sched.hdr->n_ctas[1] = gridDim.x < kMaxCtas ? gridDim.x : kMaxCtas;
    }

    // Q tiles that see key block `blk`: [first_q, n_q)
    auto q_range = [](const WorkItem& w, int& first_q, int& n_q) {
        n_q = (w.len + kTile - 1) / kTile;
        first_q = CAUSAL ? w.blk : 0;
    };

    if (warp >= 8 && warp < 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
    if (warp == 9) {
        // ------------------------------------------------- scheduler, TMA producer, statistics staging
        if (lane == 0) {
            tma_prefetch_desc(&tmap_q);
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            tma_prefetch_desc(&tmap_do);
        }
        const uint32_t n_items = p.sched.hdr->n_items;
        uint32_t n_work = 0, g = 0;
        while (true) {
            const uint32_t slot = n_work & 1u;
            WorkItem w;
            if (lane == 0) {
                if (n_work >= 2) mbar_wait(&sh.work_empty[slot], ((n_work >> 1) - 1) & 1u, guard);
                const uint32_t item = atomicAdd(&p.sched.hdr->work_counter, 1u);
                if (item < n_items && !sh.abort_flag) {
                    w = decode_item(p.sched, p.cu_seqlens, item, kTile, p.n_heads, false);
                } else {
                    w.tok0 = 0; w.len = -1; w.head = 0; w.blk = 0; w.tile0 = 0;
                }
                sh.work[slot] = w;
                mbar_arrive(&sh.work_full[slot]);
            }
            w.tok0 = __shfl_sync(0xffffffffu, w.tok0, 0);
            w.len = __shfl_sync(0xffffffffu, w.len, 0);
            w.head = __shfl_sync(0xffffffffu, w.head, 0);
            w.blk = __shfl_sync(0xffffffffu, w.blk, 0);
            if (w.len < 0) break;
            int first_q, n_q;
            q_range(w, first_q, n_q);
            if (lane == 0) {
                if (n_work >= 1) mbar_wait(&sh.kv_empty, (n_work - 1) & 1u, guard);
                mbar_expect_tx(&sh.kv_full, 2 * Cfg::kTileBytes);
                bwd_load_tile<D>(smem + Cfg::kOffK, &tmap_k, &sh.kv_full, w.head, w.tok0 + w.blk * kTile);
                bwd_load_tile<D>(smem + Cfg::kOffV, &tmap_v, &sh.kv_full, w.head, w.tok0 + w.blk * kTile);
            }
            ++n_work;
            for (int i = first_q; i < n_q; ++i, ++g) {
                const uint32_t stage = g % Cfg::kQStages, fill = g / Cfg::kQStages;
                const int row = w.tok0 + i * kTile;
                if (lane == 0) {
                    if (fill >= 1) mbar_wait(&sh.q_empty[stage], (fill - 1) & 1u, guard);
                    mbar_expect_tx(&sh.q_full[stage], Cfg::kTileBytes);
                    bwd_load_tile<D>(smem + Cfg::kOffQ + stage * Cfg::kTileBytes, &tmap_q, &sh.q_full[stage], w.head, row);
                    // per-query terms (2 slots): slot g&1 is free once the rank-1 MMAs of tile g-2 are done.
                    // The 4 KB block of this (tile, head) comes by bulk copy in the layout the MMA reads.
                    if (g >= 2) mbar_wait(&sh.stat_empty[g & 1u], ((g >> 1) - 1) & 1u, guard);
                    mbar_expect_tx(&sh.stat_full[g & 1u], Cfg::kStatBytes);
                    tma_load_bulk(smem + Cfg::kOffStat + (g & 1u) * Cfg::kStatBytes,
                                  p.stats + (((size_t)w.tile0 + i) * p.n_heads + w.head) * (Cfg::kStatBytes / 2),
                                  Cfg::kStatBytes, &sh.stat_full[g & 1u]);
                    if (g >= 1) mbar_wait(&sh.do_empty, (g - 1) & 1u, guard);
                    mbar_expect_tx(&sh.do_full, Cfg::kTileBytes);
                    bwd_load_tile<D>(smem + Cfg::kOffDo, &tmap_do, &sh.do_full, w.head, row);
                }
            }
        }
    } else if (warp == 8) {
        // ------------------------------------------------- MMA issue
        // All 32 lanes run the loop in lock step and only `leader` issues, so that every operand is
        // warp-uniform and an MMA costs a couple of adds: each instruction between two MMAs is pipe idle time.
        {
            const bool leader = elect_one();
            // Shared-memory descriptors are built once; a k-step only adds a constant to the address
            // field (the issuing thread is on the critical path: MMA issue blocks while the pipe is busy).
            constexpr uint32_t idesc_abt = make_idesc_bf16(128, 128, false, false);  // both operands K-contiguous
            const int n_ks = TRIM ? (p.head_dim + 15) >> 4 : D / 16;                // steps of 16 head_dim columns that hold data
            const uint32_t idesc_nd_kb = make_idesc_bf16(128, TRIM ? n_ks * 16 : D, false, true);   // A K-contig / tmem, B N-contig
            const uint32_t idesc_nd_mm = make_idesc_bf16(128, TRIM ? n_ks * 16 : D, true, true);    // A M-contig, B N-contig
            constexpr uint32_t kStageStep = Cfg::kTileBytes >> 4;
            const uint64_t k_km = make_sdesc_sw128(smem_u32(smem + Cfg::kOffK), 16, 1024);
            const uint64_t k_mn = make_sdesc_sw128(smem_u32(smem + Cfg::kOffK), Cfg::kBoxBytes, 1024);
            const uint64_t v_km = make_sdesc_sw128(smem_u32(smem + Cfg::kOffV), 16, 1024);
            const uint64_t q_km0 = make_sdesc_sw128(smem_u32(smem + Cfg::kOffQ), 16, 1024);
            const uint64_t q_mn0 = make_sdesc_sw128(smem_u32(smem + Cfg::kOffQ), Cfg::kBoxBytes, 1024);
            const uint64_t do_km = make_sdesc_sw128(smem_u32(smem + Cfg::kOffDo), 16, 1024);
            const uint64_t do_mn = make_sdesc_sw128(smem_u32(smem + Cfg::kOffDo), Cfg::kBoxBytes, 1024);
            const uint64_t ds_km = make_sdesc_sw128(smem_u32(smem + Cfg::kOffDs), 16, 1024);
            const uint64_t ds_mn = make_sdesc_sw128(smem_u32(smem + Cfg::kOffDs), 16384, 1024);
            const uint64_t ones_s = make_sdesc_nosw(smem_u32(smem + Cfg::kOffOnes), 2048, 128);
            const uint64_t ones_d = make_sdesc_nosw(smem_u32(smem + Cfg::kOffOnes + Cfg::kStatBytes), 2048, 128);
            const uint64_t stat0 = make_sdesc_nosw(smem_u32(smem + Cfg::kOffStat), 2048, 128);
            constexpr uint32_t kStatStep = Cfg::kStatBytes >> 4;
            // address-field increments (16-byte units) of k-step ks
            auto km_step = [](int ks, int box_bytes) -> uint64_t { return (uint64_t)(((ks / 4) * box_bytes + (ks % 4) * 32) >> 4); };
            auto mn_step = [](int ks) -> uint64_t { return (uint64_t)((ks * 2048) >> 4); };
            // D[128 x 128] = A B^T, both [128 x D] tiles with head_dim contiguous
            auto issue_abt = [&](uint32_t d_tmem, uint64_t a, uint64_t b) {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    if (leader && (!TRIM || ks < n_ks))
                        tc_mma_ss(d_tmem, a + km_step(ks, Cfg::kBoxBytes), b + km_step(ks, Cfg::kBoxBytes), idesc_abt, ks > 0);
            };
            uint32_t n_work = 0, g = 0;
            while (true) {
                const uint32_t slot = n_work & 1u;
                const bool got = mbar_wait(&sh.work_full[slot], (n_work >> 1) & 1u, guard);
                if (!__all_sync(0xffffffffu, got)) break;
                const WorkItem w = sh.work[slot];
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.work_empty[slot]);
                if (w.len < 0) break;
                int first_q, n_q;
                q_range(w, first_q, n_q);
                const int N = n_q - first_q;
                mbar_wait(&sh.kv_full, n_work & 1u, guard);
                // S^T and dP^T of the first tile
                uint32_t stage = g % Cfg::kQStages;
                mbar_wait(&sh.q_full[stage], (g / Cfg::kQStages) & 1u, guard);
                tc_fence_after();
                mbar_wait(&sh.stat_full[g & 1u], (g >> 1) & 1u, guard);
                issue_abt(tmem + Cfg::kSt, k_km, q_km0 + stage * kStageStep);
                if (leader) tc_mma_ss(tmem + Cfg::kSt, ones_s, stat0 + (g & 1u) * kStatStep, idesc_abt, true);
                if (leader) tc_commit(&sh.s_full);
                mbar_wait(&sh.do_full, g & 1u, guard);
                if (g >= 1) mbar_wait(&sh.dq_free, (g - 1) & 1u, guard);
                tc_fence_after();
                issue_abt(tmem + Cfg::kDp, v_km, do_km);
                if (leader) tc_mma_ss(tmem + Cfg::kDp, ones_d, stat0 + (g & 1u) * kStatStep, idesc_abt, true);
                if (leader) tc_commit(&sh.dp_full);
                if (leader) tc_commit(&sh.stat_empty[g & 1u]);
                for (int n = 0; n < N; ++n, ++g) {
                    const uint32_t nstage = stage + 1 == Cfg::kQStages ? 0 : stage + 1;
                    const bool has_next = n + 1 < N;
                    // dV += P^T dO
                    mbar_wait(&sh.p_half, g & 1u, guard);
                    if (n == 0 && n_work >= 1) mbar_wait(&sh.dkv_free, (n_work - 1) & 1u, guard);
                    tc_fence_after();
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        if (part == 1) {
                            mbar_wait(&sh.p_full, g & 1u, guard);
                            tc_fence_after();
                        }
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int ks = (k4 / 2) * 4 + part * 2 + (k4 % 2);     // k-steps {0,1,4,5} then {2,3,6,7}
                            if (leader) tc_mma_ts(tmem + Cfg::kDv, tmem + Cfg::kSt + (ks / 4) * 64 + (ks % 4) * 8, do_mn + mn_step(ks),
                                      idesc_nd_kb, n > 0 || part > 0 || k4 > 0);
                        }
                    }
                    if (leader) tc_commit(&sh.do_empty);
                    // S^T of the next tile
                    if (has_next) {
                        mbar_wait(&sh.q_full[nstage], ((g + 1) / Cfg::kQStages) & 1u, guard);
                        mbar_wait(&sh.stat_full[(g + 1) & 1u], ((g + 1) >> 1) & 1u, guard);
                        tc_fence_after();
                        issue_abt(tmem + Cfg::kSt, k_km, q_km0 + nstage * kStageStep);
                        if (leader) tc_mma_ss(tmem + Cfg::kSt, ones_s, stat0 + ((g + 1) & 1u) * kStatStep, idesc_abt, true);
                        if (leader) tc_commit(&sh.s_full);
                    }
                    // dQ tile = dS K  (A: dS^T read M-contiguous; B: K with head_dim contiguous)
                    mbar_wait(&sh.ds_full, g & 1u, guard);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kTile / 16; ++ks)
                        if (leader) tc_mma_ss(tmem + Cfg::kDp, ds_mn + mn_step(ks), k_mn + mn_step(ks), idesc_nd_mm, ks > 0);
                    if (leader) tc_commit(&sh.dq_full);
                    // dK += dS^T Q
#pragma unroll
                    for (int ks = 0; ks < kTile / 16; ++ks)
                        if (leader) tc_mma_ss(tmem + Cfg::kDk, ds_km + km_step(ks, 16384), q_mn0 + stage * kStageStep + mn_step(ks),
                                  idesc_nd_kb, n > 0 || ks > 0);
                    if (leader) tc_commit(&sh.q_empty[stage]);
                    if (leader) tc_commit(&sh.ds_free);
                    // dP^T of the next tile (its columns hold dQ until the drain warps have read it)
                    if (has_next) {
                        mbar_wait(&sh.do_full, (g + 1) & 1u, guard);
                        mbar_wait(&sh.dq_free, g & 1u, guard);
                        tc_fence_after();
                        issue_abt(tmem + Cfg::kDp, v_km, do_km);
                        if (leader) tc_mma_ss(tmem + Cfg::kDp, ones_d, stat0 + ((g + 1) & 1u) * kStatStep, idesc_abt, true);
                        if (leader) tc_commit(&sh.dp_full);
                        if (leader) tc_commit(&sh.stat_empty[(g + 1) & 1u]);
                    }
                    stage = nstage;
                }
                if (leader) tc_commit(&sh.dkv_full);
                if (leader) tc_commit(&sh.kv_empty);
                ++n_work;
            }
        }
    }
    } else if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 136;");
        // ------------------------------------------------- compute: P^T, dS^T, final dK / dV
        const int half = warp >> 2;                                  // which 64 query columns
        const int key_in_tile = (warp & 3) * 32 + lane;              // tensor-memory lane = key
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t st_tmem = tmem + lane_base + Cfg::kSt + half * 64;
        const uint32_t pt_tmem = tmem + lane_base + Cfg::kSt + half * 64;   // bf16 pairs, inside this group's own S^T columns
        const uint32_t dp_tmem = tmem + lane_base + Cfg::kDp + half * 64;
        uint8_t* ds_row = smem + Cfg::kOffDs + half * 16384;
        uint32_t n_work = 0, g = 0, n_staged = 0;
        while (true) {
            const uint32_t slot = n_work & 1u;
            const bool got = mbar_wait(&sh.work_full[slot], (n_work >> 1) & 1u, guard);
            if (!__all_sync(0xffffffffu, got)) break;
            const WorkItem w = sh.work[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.work_empty[slot]);
            if (w.len < 0) break;
            int first_q, n_q;
            q_range(w, first_q, n_q);
            const int key = w.blk * kTile + key_in_tile;
            const bool key_valid = key < w.len;
            const bool key_tail = (w.blk + 1) * kTile > w.len;

            if (p.bounds != nullptr && w.len <= kTile) {     // one tile pair, possibly several merged sequences
                compute_single_tile_item<CAUSAL>(sh, p, w, st_tmem, dp_tmem, ds_row, half, key_in_tile, g, guard);
                ++g;
                first_q = n_q;                                // nothing left for the loop below
            }
            for (int i = first_q; i < n_q; ++i, ++g) {
                const bool diag = CAUSAL && i == w.blk;
                float pf[64];
                mbar_wait(&sh.s_full, g & 1u, guard);
                tc_fence_after();
                {
                    // all 64 scores of this thread's key row are requested before the single wait
                    uint32_t sr[64];
                    tmem_ld_x32(st_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                    tmem_ld_x32(st_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        // 32 query columns at a time: the dV product starts on the first chunk while the
                        // second is still being exponentiated
#pragma unroll
                        for (int e = 0; e < 32; ++e) pf[c * 32 + e] = fast_exp2(__uint_as_float(sr[c * 32 + e]) * p.scale_log2);
                        if (key_tail || diag) {
                            const int q_first = i * kTile + half * 64 + c * 32;   // query index of element 0
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (!key_valid || (diag && key > q_first + e)) pf[c * 32 + e] = 0.f;
                        }
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) pk[e] = pack_bf16x2(pf[c * 32 + 2 * e], pf[c * 32 + 2 * e + 1]);
                        tmem_st_x16(pt_tmem + c * 16, pk);
                        if (c == 0) {
                            tmem_wait_st();
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sh.p_half);
                        }
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.p_full);

                // dS^T = P^T o (dP^T - D)
                mbar_wait(&sh.dp_full, g & 1u, guard);
                if (g >= 1) mbar_wait(&sh.ds_free, (g - 1) & 1u, guard);
                tc_fence_after();
                {
                    uint32_t dr[64];
                    tmem_ld_x32(dp_tmem, *reinterpret_cast<uint32_t(*)[32]>(&dr[0]));
                    tmem_ld_x32(dp_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&dr[32]));
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            pk[e] = pack_bf16x2(pf[c * 8 + 2 * e] * __uint_as_float(dr[c * 8 + 2 * e]),
                                                pf[c * 8 + 2 * e + 1] * __uint_as_float(dr[c * 8 + 2 * e + 1]));
                        *reinterpret_cast<uint4*>(ds_row + sw128_offset(key_in_tile, c)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                fence_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.ds_full);
            }

            // item epilogue: dV and dK rows of this key block (each group writes half the columns)
            mbar_wait(&sh.dkv_full, n_work & 1u, guard);
            tc_fence_after();
            if (D == 128 && w.blk * kTile + kTile <= w.len) {
                store_dkv_staged<D>(sh, &tmap_dk, &tmap_dv, smem + Cfg::kOffDs + half * 16384, tmem + lane_base, half, w.head,
                                    w.tok0 + w.blk * kTile, p.scale, n_staged, guard);
                n_staged += 2;
                ++n_work;
                continue;
            }
            const size_t tok = (size_t)w.tok0 + (size_t)key;
            const size_t out_off = tok * p.row_stride + w.head * p.head_dim + half * (D / 2);
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t src = tmem + lane_base + (which == 0 ? Cfg::kDv : Cfg::kDk) + half * (D / 2);
                __nv_bfloat16* dst = (which == 0 ? p.dv : p.dk) + out_off;
                const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t acc[32];
                    tmem_ld_x32(src + c * 32, acc);
                    tmem_wait_ld();
                    if (key_valid) {
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint4 val;
                            val.x = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 0]) * mul, __uint_as_float(acc[v4 * 8 + 1]) * mul);
                            val.y = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 2]) * mul, __uint_as_float(acc[v4 * 8 + 3]) * mul);
                            val.z = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 4]) * mul, __uint_as_float(acc[v4 * 8 + 5]) * mul);
                            val.w = pack_bf16x2(__uint_as_float(acc[v4 * 8 + 6]) * mul, __uint_as_float(acc[v4 * 8 + 7]) * mul);
                            if (half * (D / 2) + c * 32 + v4 * 8 < p.head_dim) *reinterpret_cast<uint4*>(dst + c * 32 + v4 * 8) = val;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.dkv_free);
            ++n_work;
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 136;");
        // ------------------------------------------------- dQ drain: tensor memory -> fp32 atomics
        const int q_in_tile = (warp & 3) * 32 + lane;               // warps 12-15 -> lane quarters 0-3
        const uint32_t dq_tmem = tmem + ((uint32_t)((warp & 3) * 32) << 16) + Cfg::kDp;
        uint32_t n_work = 0, g = 0;
        while (true) {
            const uint32_t slot = n_work & 1u;
            const bool got = mbar_wait(&sh.work_full[slot], (n_work >> 1) & 1u, guard);
            if (!__all_sync(0xffffffffu, got)) break;
            const WorkItem w = sh.work[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.work_empty[slot]);
            if (w.len < 0) break;
            ++n_work;
            int first_q, n_q;
            q_range(w, first_q, n_q);
            for (int i = first_q; i < n_q; ++i, ++g) {
                mbar_wait(&sh.dq_full, g & 1u, guard);
                tc_fence_after();
                // accumulator block of (tile, head) is [D/4][128 rows][4]: the 32 rows of a warp are
                // contiguous for a fixed column group, so each vector atomic covers whole sectors
                const int qrow = i * kTile + q_in_tile;
                float* dst = p.dq_acc + (((size_t)w.tile0 + i) * p.n_heads + w.head) * (size_t)(kTile * D) + q_in_tile * 4;
                // read the whole tile first and release tensor memory at once: dP^T of the next tile waits
                // on it, while the atomics below may take as long as they like
                uint32_t acc[D];
#pragma unroll
                for (int c = 0; c < D / 32; ++c) tmem_ld_x32(dq_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[c * 32]));
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.dq_free);
                if (w.len <= kTile) {
                    // the sequence's only tile pair: this is the whole dQ, no accumulation needed
                    if (qrow < w.len) {
                        __nv_bfloat16* out = p.dq + ((size_t)w.tok0 + qrow) * p.row_stride + w.head * p.head_dim;
#pragma unroll
                        for (int c = 0; c < D / 8; ++c) {
                            uint4 val;
                            val.x = pack_bf16x2(__uint_as_float(acc[c * 8 + 0]) * p.scale, __uint_as_float(acc[c * 8 + 1]) * p.scale);
                            val.y = pack_bf16x2(__uint_as_float(acc[c * 8 + 2]) * p.scale, __uint_as_float(acc[c * 8 + 3]) * p.scale);
                            val.z = pack_bf16x2(__uint_as_float(acc[c * 8 + 4]) * p.scale, __uint_as_float(acc[c * 8 + 5]) * p.scale);
                            val.w = pack_bf16x2(__uint_as_float(acc[c * 8 + 6]) * p.scale, __uint_as_float(acc[c * 8 + 7]) * p.scale);
                            if (c * 8 < p.head_dim) *reinterpret_cast<uint4*>(out + c * 8) = val;
                        }
                    }
                } else {
                    const bool live = qrow < w.len;
                    if ((warp & 3) > 0) __nanosleep((warp & 3) * kRedStaggerNs + 64);
                    const int n_c4 = TRIM ? ((p.head_dim + 15) >> 4) * 4 : D / 4;     // groups of four columns that hold data
#pragma unroll
                    for (int c = 0; c < D / 4; ++c) {
                        if (TRIM && c >= n_c4) break;
                        if (live) red_add_v4(dst + c * (kTile * 4), __uint_as_float(acc[c * 4]), __uint_as_float(acc[c * 4 + 1]),
                                   __uint_as_float(acc[c * 4 + 2]), __uint_as_float(acc[c * 4 + 3]));
                        if ((c % kRedGroup) == kRedGroup - 1) __nanosleep(kRedSleepNs);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && blockIdx.x < kMaxCtas) p.sched.spans[1 * kMaxCtas + blockIdx.x].end_ns = global_timer_ns();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int D, bool CAUSAL, bool TRIM>
static cudaError_t launch_one(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                              const CUtensorMap& tdk, const CUtensorMap& tdv, const BwdParams& p, int n_ctas, cudaStream_t stream) {
    auto kern = attn_bwd_kernel<D, CAUSAL, TRIM>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<D>::kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<n_ctas, kBwdThreads, BwdCfg<D>::kSmemBytes, stream>>>(tq, tk, tv, tdo, tdk, tdv, p);
    return cudaGetLastError();
}

cudaError_t launch_attn_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                            const CUtensorMap& tdk, const CUtensorMap& tdv, const BwdParams& p, int head_dim, bool causal,
                            int n_ctas, cudaStream_t stream) {
    if (head_dim > 112)
        return causal ? launch_one<128, true, false>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream)
                      : launch_one<128, false, false>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream);
    if (head_dim > 64)
        return causal ? launch_one<128, true, true>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream)
                      : launch_one<128, false, true>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream);
    return causal ? launch_one<64, true, false>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream)
                  : launch_one<64, false, false>(tq, tk, tv, tdo, tdk, tdv, p, n_ctas, stream);
}

}  // namespace dcp
