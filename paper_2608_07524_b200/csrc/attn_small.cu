// Attention for batches in which EVERY sequence is very short (at most 32 tokens): the temporal axis of a
// 2-D model (Section 4.1 of the paper: sequences of a handful of frames, tens of thousands of them).
//
// Such a batch is bound by HBM, not by the tensor cores: a sequence of L tokens moves 4 L d bytes per head
// and needs 4 L^2 d flops, a ratio of L flops per byte.  What matters is bytes in flight per SM and
// instructions per byte, not MMA shape: the 128-row tile kernels expose a load's latency once per tile.
//
// Here every WARP runs its own two-stage pipeline, with no CTA-wide barrier: the packed batch is cut into
// chunks of `chunk` consecutive token positions, a work item is (chunk, head) and covers the sequences that
// start in the chunk, and warps take items round robin (items are equal in tokens by construction, so a
// static assignment balances).  A warp cuts an item's sequences into runs of consecutive sequences of at
// most 16 (32) rows together, fetches exactly a run's rows of q, k, v (dO, lse) with asynchronous 16-byte
// copies into one of its two stages, and while those arrive computes the previous run in registers with
// warp-level MMAs (16x8x16; the tiles are far too small for a 128-row tensor-memory accumulator), every row
// masked to the keys of its own sequence.  Results are staged in the shared-memory rows of operands that are
// no longer needed and leave as 16-byte stores.  No pre or post pass: the backward forms
// D_i = sum_j P_ij dP_ij in registers (equal to sum_c dO_ic O_ic because O = P V; `o` is not read) and writes
// dq directly.
//
// Measured on 20384 sequences of 1-13 tokens, 16 heads of 128 (forward / backward, ms; the tile kernels take
// 0.52 / 1.37 with their pre and post passes, copies and stores alone 0.34 / 0.59):
//   one CTA per (sequence, four heads), one bulk copy per row         0.77 / 1.47   (copy engine: one operation per
//   the same with 16-byte asynchronous copies                         0.73 / 1.36    ~115 cycles; CTA lifetime ~6 us)
//   persistent CTAs, items of ~56 rows in two CTA-wide stages,
//     a warp per sequence, head dimension at run time                 0.67 / 1.72   (instruction issue: ~1500 per sequence)
//   head dimension at compile time, stmatrix staging                  0.51 / 0.98
//   runs of sequences per warp pass, cheaper copy loops and run search 0.46 / 0.78  (half the warps idle at each barrier)
//   this form: every warp its own pipeline                            0.34 / 0.61
#include <climits>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "attn_kernels.h"
#include "sm100_ptx.cuh"

namespace dcp {
namespace {


struct SmallParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const __nv_bfloat16* d_o;   // backward only
    __nv_bfloat16* o;           // forward only
    __nv_bfloat16* dq;          // backward only
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    float* lse;                 // written by the forward, read by the backward
    const int32_t* cu;
    const int32_t* first_seq;   // [n_chunks + 1]: first sequence starting at or after position c * chunk
    WorkspaceHeader* hdr;
    int32_t n_heads;
    int32_t head_dim;
    int32_t total_tokens;
    int32_t chunk;              // token positions per chunk
    int32_t n_chunks;
    int32_t stages;             // stages per warp: 2 (copies of the next run overlap this run) or 1 (more warps per SM)
    int32_t causal;
    int64_t row_stride;
    float scale;
    float scale_log2;
};

// ---- warp-level matrix instructions and copies ------------------------------------------------------------
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// D (16x8) += A (16x8) * B (8x8): the last 8 columns of a head dimension that is not a multiple of 16
__device__ __forceinline__ void mma_k8(float (&c)[4], const uint32_t (&a)[2], uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b0));
}
// transpose of an 8x8 block of 16-bit values held one register per lane in the fragment layout
__device__ __forceinline__ uint32_t transpose8x8(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
// global -> shared without passing through registers
__device__ __forceinline__ void copy_async_16(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void copy_async_4(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_shared_4(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// A run of consecutive sequences (at most 16 * NB rows together: one warp computes them in one pass, each row
// masked to the keys of its own sequence) inside the tiles of a stage: the row pitch, its rows, and the row of
// zeros every ldmatrix row past the run's end points at (so that a neighbour's rows or stale shared memory
// never reach a product).
struct SeqView {
    uint32_t zero, dump, pitch;     // zero: a row of zeros to read; dump: a row nobody reads, for stores of rows past the end
    int len;                        // rows of the run
    uint32_t starts;                // bit r set = a sequence of the run starts at its row r (bit 0 always)
};

// keys [lo, hi) that query row i of a run may see: the rows of its own sequence (rows past the end: any, never stored)
__device__ __forceinline__ void row_range(const SeqView& s, int i, int& lo, int& hi) {
    if (i >= s.len) {
        lo = 0;
        hi = s.len;
        return;
    }
    lo = 31 - __clz(s.starts & (0xffffffffu >> (31 - i)));
    const uint32_t later = i < 31 ? s.starts >> (i + 1) : 0u;
    hi = later ? i + __ffs(later) : s.len;
}

__device__ __forceinline__ uint32_t row_ptr(const SeqView& s, uint32_t tile, int r, uint32_t col) {
    return r < s.len ? tile + (uint32_t)r * s.pitch + col : s.zero;
}

// C (16 x 16 block: rows of `a_tile` from a_row0, rows of `b_tile` from b_row0) += A B^T over the head dimension
__device__ __forceinline__ void product_over_d(float (&c)[2][4], const SeqView& s, uint32_t a_tile, int a_row0, uint32_t b_tile,
                                               int b_row0, int d, int lane) {
    const int a_r = a_row0 + (lane & 7) + ((lane >> 3) & 1) * 8, a_c = ((lane >> 4) & 1) * 8;
    const int b_r = b_row0 + (lane & 7) + ((lane >> 4) & 1) * 8, b_c = ((lane >> 3) & 1) * 8;
    for (int k0 = 0; k0 + 16 <= d; k0 += 16) {
        uint32_t a[4], b[4];
        ldsm_x4(a, row_ptr(s, a_tile, a_r, (uint32_t)(k0 + a_c) * 2));
        ldsm_x4(b, row_ptr(s, b_tile, b_r, (uint32_t)(k0 + b_c) * 2));
        mma_k16(c[0], a, b[0], b[1]);
        mma_k16(c[1], a, b[2], b[3]);
    }
    if (d & 8) {
        const int k0 = d - 8;
        uint32_t a[2], b[2];
        ldsm_x2(a, row_ptr(s, a_tile, a_row0 + (lane & 15), (uint32_t)k0 * 2));
        ldsm_x2(b, row_ptr(s, b_tile, b_row0 + (lane & 15), (uint32_t)k0 * 2));
        mma_k8(c[0], a, b[0]);
        mma_k8(c[1], a, b[1]);
    }
}

// acc (16 rows x d columns, 8 columns per entry) += A (16 x 16 fragment) * rows [row0, row0 + 16) of `b_tile`
__device__ __forceinline__ void product_into_d(float (&acc)[16][4], const uint32_t (&a)[4], const SeqView& s, uint32_t b_tile,
                                               int row0, int d, int lane) {
    const int b_r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8, b_c = ((lane >> 4) & 1) * 8;
#pragma unroll
    for (int np = 0; np < 8; ++np) {
        if (np * 16 < d) {
            uint32_t b[4];
            const int col = np * 16 + b_c;
            ldsm_x4_t(b, col < d ? row_ptr(s, b_tile, b_r, (uint32_t)col * 2) : s.zero);
            mma_k16(acc[2 * np], a, b[0], b[1]);
            if (np * 16 + 8 < d) mma_k16(acc[2 * np + 1], a, b[2], b[3]);
        }
    }
}

// acc * mul -> bf16 into rows row0 + g and row0 + g + 8 of the sequence's rows in `tile`; rows past its end skipped
__device__ __forceinline__ void stage_rows(const float (&acc)[16][4], float mul0, float mul1, const SeqView& s, uint32_t tile, int row0,
                                           int d, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const uint32_t base = tile + (uint32_t)t * 4;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
        if (nt * 8 < d) {
            if (row0 + g < s.len)
                st_shared_4(base + (uint32_t)(row0 + g) * s.pitch + nt * 16, pack_bf16x2(acc[nt][0] * mul0, acc[nt][1] * mul0));
            if (row0 + g + 8 < s.len)
                st_shared_4(base + (uint32_t)(row0 + g + 8) * s.pitch + nt * 16, pack_bf16x2(acc[nt][2] * mul1, acc[nt][3] * mul1));
        }
    }
}

__device__ __forceinline__ float quad_max(float x) {
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
    return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
}
__device__ __forceinline__ float quad_sum(float x) {
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    return x + __shfl_xor_sync(0xffffffffu, x, 2);
}

// ---- one sequence, one warp ---------------------------------------------------------------------------------
// NB = 16-row blocks a sequence may have (1: up to 16 tokens, 2: up to 32).  q_s, k_s, v_s (g_s) = addresses of
// the sequence's first row in the tiles.  Forward: O rows take the place of the Q rows; lse goes to global.
template <int NB>
__device__ __forceinline__ void fwd_sequence(const SmallParams& p, const SeqView& s, uint32_t q_s, uint32_t k_s, uint32_t v_s,
                                             float* lse_out, int lane) {
    const int g = lane >> 2, t = lane & 3, d = p.head_dim, len = s.len;
    const int n_b = (len + 15) >> 4;
    for (int rb = 0; rb < n_b; ++rb) {
        float sc[NB][2][4];
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sc[kb][i >> 2][i & 3] = 0.f;
            if (kb < n_b) product_over_d(sc[kb], s, q_s, rb * 16, k_s, kb * 16, d, lane);
        }
        // softmax of rows i0 and i1 over the keys this lane holds, completed across the four lanes of a quad
        const int i0 = rb * 16 + g, i1 = i0 + 8;
        int lo0, hi0, lo1, hi1;
        row_range(s, i0, lo0, hi0);
        row_range(s, i1, lo1, hi1);
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int kb = 0; kb < NB; ++kb)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int j = kb * 16 + nt * 8 + 2 * t + e;
                    const float x0 = j >= lo0 && j < hi0 && (!p.causal || j <= i0) ? sc[kb][nt][e] * p.scale_log2 : -INFINITY;
                    const float x1 = j >= lo1 && j < hi1 && (!p.causal || j <= i1) ? sc[kb][nt][2 + e] * p.scale_log2 : -INFINITY;
                    sc[kb][nt][e] = x0;
                    sc[kb][nt][2 + e] = x1;
                    m0 = fmaxf(m0, x0);
                    m1 = fmaxf(m1, x1);
                }
        m0 = quad_max(m0);
        m1 = quad_max(m1);
        float l0 = 0.f, l1 = 0.f;
        uint32_t pa[NB][4];
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            float e[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                e[nt][0] = fast_exp2(sc[kb][nt][0] - m0);
                e[nt][1] = fast_exp2(sc[kb][nt][1] - m0);
                e[nt][2] = fast_exp2(sc[kb][nt][2] - m1);
                e[nt][3] = fast_exp2(sc[kb][nt][3] - m1);
                l0 += e[nt][0] + e[nt][1];
                l1 += e[nt][2] + e[nt][3];
            }
            pa[kb][0] = pack_bf16x2(e[0][0], e[0][1]);
            pa[kb][1] = pack_bf16x2(e[0][2], e[0][3]);
            pa[kb][2] = pack_bf16x2(e[1][0], e[1][1]);
            pa[kb][3] = pack_bf16x2(e[1][2], e[1][3]);
        }
        l0 = quad_sum(l0);
        l1 = quad_sum(l1);
        float acc[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
        for (int kb = 0; kb < NB; ++kb)
            if (kb < n_b) product_into_d(acc, pa[kb], s, v_s, kb * 16, d, lane);
        stage_rows(acc, 1.0f / l0, 1.0f / l1, s, q_s, rb * 16, d, lane);
        if (t == 0) {
            if (i0 < len) lse_out[i0] = (m0 + __log2f(l0)) * 0.6931471805599453f;
            if (i1 < len) lse_out[i1] = (m1 + __log2f(l1)) * 0.6931471805599453f;
        }
    }
}

// Backward: dV rows take the place of the V rows, dQ of the dO rows, dK of the K rows (each once the operand
// is no longer needed).  lse_s = the sequence's lse values (shared memory).
template <int NB>
__device__ __forceinline__ void bwd_sequence(const SmallParams& p, const SeqView& s, uint32_t q_s, uint32_t k_s, uint32_t v_s,
                                             uint32_t g_s, const float* lse_s, int lane) {
    const int g = lane >> 2, t = lane & 3, d = p.head_dim, len = s.len;
    const int n_b = (len + 15) >> 4;
    // P and dS of every 16 x 16 block as bf16 A fragments (rows = queries, columns = keys)
    uint32_t pa[NB][NB][4], dsa[NB][NB][4];
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
        if (rb < n_b) {
            const int i0 = rb * 16 + g, i1 = i0 + 8;
            int lo0, hi0, lo1, hi1;
            row_range(s, i0, lo0, hi0);
            row_range(s, i1, lo1, hi1);
            const float lse0 = i0 < len ? lse_s[i0] * 1.4426950408889634f : 0.f;
            const float lse1 = i1 < len ? lse_s[i1] * 1.4426950408889634f : 0.f;
            float pr[NB][2][4], dp[NB][2][4];
            float d0 = 0.f, d1 = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb) {
#pragma unroll
                for (int i = 0; i < 8; ++i) pr[kb][i >> 2][i & 3] = dp[kb][i >> 2][i & 3] = 0.f;
                if (kb < n_b) {
                    product_over_d(pr[kb], s, q_s, rb * 16, k_s, kb * 16, d, lane);
                    product_over_d(dp[kb], s, g_s, rb * 16, v_s, kb * 16, d, lane);
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int j = kb * 16 + nt * 8 + 2 * t + e;
                        const bool v0 = j >= lo0 && j < hi0 && i0 < len && (!p.causal || j <= i0);
                        const bool v1 = j >= lo1 && j < hi1 && i1 < len && (!p.causal || j <= i1);
                        const float p0 = v0 ? fast_exp2(pr[kb][nt][e] * p.scale_log2 - lse0) : 0.f;
                        const float p1 = v1 ? fast_exp2(pr[kb][nt][2 + e] * p.scale_log2 - lse1) : 0.f;
                        pr[kb][nt][e] = p0;
                        pr[kb][nt][2 + e] = p1;
                        d0 += p0 * dp[kb][nt][e];
                        d1 += p1 * dp[kb][nt][2 + e];
                    }
            }
            d0 = quad_sum(d0);
            d1 = quad_sum(d1);
#pragma unroll
            for (int kb = 0; kb < NB; ++kb) {
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    pa[rb][kb][nt * 2 + 0] = pack_bf16x2(pr[kb][nt][0], pr[kb][nt][1]);
                    pa[rb][kb][nt * 2 + 1] = pack_bf16x2(pr[kb][nt][2], pr[kb][nt][3]);
                    dsa[rb][kb][nt * 2 + 0] = pack_bf16x2(pr[kb][nt][0] * (dp[kb][nt][0] - d0), pr[kb][nt][1] * (dp[kb][nt][1] - d0));
                    dsa[rb][kb][nt * 2 + 1] = pack_bf16x2(pr[kb][nt][2] * (dp[kb][nt][2] - d1), pr[kb][nt][3] * (dp[kb][nt][3] - d1));
                }
            }
        } else {
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
#pragma unroll
                for (int i = 0; i < 4; ++i) pa[rb][kb][i] = dsa[rb][kb][i] = 0u;
        }
    }

    float acc[16][4];
    // dV (keys kb) = sum over query blocks of P^T dO
#pragma unroll
    for (int kb = 0; kb < NB; ++kb) {
        if (kb < n_b) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int rb = 0; rb < NB; ++rb) {
                if (rb < n_b) {
                    const uint32_t at[4] = {transpose8x8(pa[rb][kb][0]), transpose8x8(pa[rb][kb][2]), transpose8x8(pa[rb][kb][1]),
                                            transpose8x8(pa[rb][kb][3])};
                    product_into_d(acc, at, s, g_s, rb * 16, d, lane);
                }
            }
            stage_rows(acc, 1.f, 1.f, s, v_s, kb * 16, d, lane);
        }
    }
    __syncwarp();
    // dQ (queries rb) = scale * sum over key blocks of dS K
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
        if (rb < n_b) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
                if (kb < n_b) product_into_d(acc, dsa[rb][kb], s, k_s, kb * 16, d, lane);
            stage_rows(acc, p.scale, p.scale, s, g_s, rb * 16, d, lane);
        }
    }
    __syncwarp();
    // dK (keys kb) = scale * sum over query blocks of dS^T Q
#pragma unroll
    for (int kb = 0; kb < NB; ++kb) {
        if (kb < n_b) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int rb = 0; rb < NB; ++rb) {
                if (rb < n_b) {
                    const uint32_t at[4] = {transpose8x8(dsa[rb][kb][0]), transpose8x8(dsa[rb][kb][2]), transpose8x8(dsa[rb][kb][1]),
                                            transpose8x8(dsa[rb][kb][3])};
                    product_into_d(acc, at, s, q_s, rb * 16, d, lane);
                }
            }
            stage_rows(acc, p.scale, p.scale, s, k_s, kb * 16, d, lane);
        }
    }
}

// ---- one sequence, one warp, head dimension known at compile time ------------------------------------------------
// Everything is unrolled and every ldmatrix / stmatrix address is a per-lane base plus a constant: the per-lane
// row (and whether it lies past the sequence end) is fixed for a whole sequence.  Measured on the temporal-axis
// workload, the form with a run-time head dimension spends 2.0 (forward) and 2.9 (backward) times the memory
// time in instruction issue; this one is what makes the kernels bound by HBM.
__device__ __forceinline__ void stsm_x4(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
// lane's row for the A operand, the transposed B operand and stmatrix: rows 0-7, 8-15 | 0-7, 8-15 ; columns +0 | +8
__device__ __forceinline__ uint32_t lane_row_a(uint32_t tile, int blk, const SeqView& s, int lane, uint32_t other) {
    const int r = blk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    return (r < s.len ? tile + (uint32_t)r * s.pitch : other) + ((lane >> 4) & 1) * 16;
}
// lane's row for the B operand read as stored (keys x d): rows 0-7, 0-7 | 8-15, 8-15 ; columns +0, +8 | +0, +8
__device__ __forceinline__ uint32_t lane_row_b(uint32_t tile, int blk, const SeqView& s, int lane) {
    const int r = blk * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
    return (r < s.len ? tile + (uint32_t)r * s.pitch : s.zero) + ((lane >> 3) & 1) * 16;
}
__device__ __forceinline__ uint32_t lane_row_tail(uint32_t tile, int blk, const SeqView& s, int lane, int d) {
    const int r = blk * 16 + (lane & 15);
    return (r < s.len ? tile + (uint32_t)r * s.pitch : s.zero) + (uint32_t)(d - 8) * 2;
}

// c (16 x 16) += A B^T over D columns; a_addr from lane_row_a, b_addr from lane_row_b
template <int D>
__device__ __forceinline__ void fast_over_d(float (&c)[2][4], uint32_t a_addr, uint32_t b_addr, uint32_t a_tail, uint32_t b_tail) {
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t a[4], b[4];
        ldsm_x4(a, a_addr + ks * 32);
        ldsm_x4(b, b_addr + ks * 32);
        mma_k16(c[0], a, b[0], b[1]);
        mma_k16(c[1], a, b[2], b[3]);
    }
    if (D % 16) {
        uint32_t a[2], b[2];
        ldsm_x2(a, a_tail);
        ldsm_x2(b, b_tail);
        mma_k8(c[0], a, b[0]);
        mma_k8(c[1], a, b[1]);
    }
}

// acc (16 x D) += A (fragment) * 16 rows of a tile read transposed; b_addr from lane_row_a
template <int D>
__device__ __forceinline__ void fast_into_d(float (&acc)[(D + 15) / 16 * 2][4], const uint32_t (&a)[4], uint32_t b_addr) {
#pragma unroll
    for (int np = 0; np < (D + 15) / 16; ++np) {
        uint32_t b[4];
        ldsm_x4_t(b, b_addr + np * 32);     // with D % 16 == 8 the last load's second half reads the row's padding: unused
        mma_k16(acc[2 * np], a, b[0], b[1]);
        if (np * 16 + 8 < D) mma_k16(acc[2 * np + 1], a, b[2], b[3]);
    }
}

// acc -> bf16 rows of a tile; st_addr from lane_row_a with the dump row (the padding takes the unused half of an odd tail)
template <int D>
__device__ __forceinline__ void fast_stage(const float (&acc)[(D + 15) / 16 * 2][4], uint32_t st_addr) {
#pragma unroll
    for (int np = 0; np < (D + 15) / 16; ++np)
        stsm_x4(st_addr + np * 32, pack_bf16x2(acc[2 * np][0], acc[2 * np][1]), pack_bf16x2(acc[2 * np][2], acc[2 * np][3]),
                pack_bf16x2(acc[2 * np + 1][0], acc[2 * np + 1][1]), pack_bf16x2(acc[2 * np + 1][2], acc[2 * np + 1][3]));
}

template <int D, int NB>
__device__ __forceinline__ void fwd_sequence_fast(const SmallParams& p, const SeqView& s, uint32_t q_s, uint32_t k_s, uint32_t v_s,
                                                  float* lse_out, int lane) {
    const int g = lane >> 2, t = lane & 3, len = s.len;
    const int n_b = (len + 15) >> 4;
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
        if (rb < n_b) {
            float sc[NB][2][4];
            const uint32_t qa = lane_row_a(q_s, rb, s, lane, s.zero), qt = lane_row_tail(q_s, rb, s, lane, D);
#pragma unroll
            for (int kb = 0; kb < NB; ++kb) {
#pragma unroll
                for (int i = 0; i < 8; ++i) sc[kb][i >> 2][i & 3] = 0.f;
                if (kb < n_b) fast_over_d<D>(sc[kb], qa, lane_row_b(k_s, kb, s, lane), qt, lane_row_tail(k_s, kb, s, lane, D));
            }
            const int i0 = rb * 16 + g, i1 = i0 + 8;
            int lo0, hi0, lo1, hi1;
            row_range(s, i0, lo0, hi0);
            row_range(s, i1, lo1, hi1);
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int j = kb * 16 + nt * 8 + 2 * t + e;
                        const float x0 = j >= lo0 && j < hi0 && (!p.causal || j <= i0) ? sc[kb][nt][e] * p.scale_log2 : -INFINITY;
                        const float x1 = j >= lo1 && j < hi1 && (!p.causal || j <= i1) ? sc[kb][nt][2 + e] * p.scale_log2 : -INFINITY;
                        sc[kb][nt][e] = x0;
                        sc[kb][nt][2 + e] = x1;
                        m0 = fmaxf(m0, x0);
                        m1 = fmaxf(m1, x1);
                    }
            m0 = quad_max(m0);
            m1 = quad_max(m1);
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    sc[kb][nt][0] = fast_exp2(sc[kb][nt][0] - m0);
                    sc[kb][nt][1] = fast_exp2(sc[kb][nt][1] - m0);
                    sc[kb][nt][2] = fast_exp2(sc[kb][nt][2] - m1);
                    sc[kb][nt][3] = fast_exp2(sc[kb][nt][3] - m1);
                    l0 += sc[kb][nt][0] + sc[kb][nt][1];
                    l1 += sc[kb][nt][2] + sc[kb][nt][3];
                }
            l0 = quad_sum(l0);
            l1 = quad_sum(l1);
            // P is normalised before the product (one rounding to bf16 either way), so O needs no scaling afterwards
            const float r0 = 1.0f / l0, r1 = 1.0f / l1;
            float acc[(D + 15) / 16 * 2][4];
#pragma unroll
            for (int nt = 0; nt < (D + 15) / 16 * 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb) {
                if (kb < n_b) {
                    const uint32_t pa[4] = {pack_bf16x2(sc[kb][0][0] * r0, sc[kb][0][1] * r0), pack_bf16x2(sc[kb][0][2] * r1, sc[kb][0][3] * r1),
                                            pack_bf16x2(sc[kb][1][0] * r0, sc[kb][1][1] * r0), pack_bf16x2(sc[kb][1][2] * r1, sc[kb][1][3] * r1)};
                    fast_into_d<D>(acc, pa, lane_row_a(v_s, kb, s, lane, s.zero));
                }
            }
            fast_stage<D>(acc, lane_row_a(q_s, rb, s, lane, s.dump));
            if (t == 0) {
                if (i0 < len) lse_out[i0] = (m0 + __log2f(l0)) * 0.6931471805599453f;
                if (i1 < len) lse_out[i1] = (m1 + __log2f(l1)) * 0.6931471805599453f;
            }
        }
    }
}

template <int D, int NB>
__device__ __forceinline__ void bwd_sequence_fast(const SmallParams& p, const SeqView& s, uint32_t q_s, uint32_t k_s, uint32_t v_s,
                                                  uint32_t g_s, const float* lse_s, int lane) {
    const int g = lane >> 2, t = lane & 3, len = s.len;
    const int n_b = (len + 15) >> 4;
    uint32_t pa[NB][NB][4], dsa[NB][NB][4];      // P and scale * dS of every block as bf16 A fragments
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
        if (rb < n_b) {
            const int i0 = rb * 16 + g, i1 = i0 + 8;
            int lo0, hi0, lo1, hi1;
            row_range(s, i0, lo0, hi0);
            row_range(s, i1, lo1, hi1);
            const float lse0 = i0 < len ? lse_s[i0] * 1.4426950408889634f : 0.f;
            const float lse1 = i1 < len ? lse_s[i1] * 1.4426950408889634f : 0.f;
            const uint32_t qa = lane_row_a(q_s, rb, s, lane, s.zero), qt = lane_row_tail(q_s, rb, s, lane, D);
            const uint32_t ga = lane_row_a(g_s, rb, s, lane, s.zero), gt = lane_row_tail(g_s, rb, s, lane, D);
            float pr[NB][2][4], dp[NB][2][4];
            float d0 = 0.f, d1 = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb) {
#pragma unroll
                for (int i = 0; i < 8; ++i) pr[kb][i >> 2][i & 3] = dp[kb][i >> 2][i & 3] = 0.f;
                if (kb < n_b) {
                    fast_over_d<D>(pr[kb], qa, lane_row_b(k_s, kb, s, lane), qt, lane_row_tail(k_s, kb, s, lane, D));
                    fast_over_d<D>(dp[kb], ga, lane_row_b(v_s, kb, s, lane), gt, lane_row_tail(v_s, kb, s, lane, D));
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int j = kb * 16 + nt * 8 + 2 * t + e;
                        const bool v0 = j >= lo0 && j < hi0 && i0 < len && (!p.causal || j <= i0);
                        const bool v1 = j >= lo1 && j < hi1 && i1 < len && (!p.causal || j <= i1);
                        const float p0 = v0 ? fast_exp2(pr[kb][nt][e] * p.scale_log2 - lse0) : 0.f;
                        const float p1 = v1 ? fast_exp2(pr[kb][nt][2 + e] * p.scale_log2 - lse1) : 0.f;
                        pr[kb][nt][e] = p0;
                        pr[kb][nt][2 + e] = p1;
                        d0 += p0 * dp[kb][nt][e];
                        d1 += p1 * dp[kb][nt][2 + e];
                    }
            }
            d0 = quad_sum(d0);
            d1 = quad_sum(d1);
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    pa[rb][kb][nt * 2 + 0] = pack_bf16x2(pr[kb][nt][0], pr[kb][nt][1]);
                    pa[rb][kb][nt * 2 + 1] = pack_bf16x2(pr[kb][nt][2], pr[kb][nt][3]);
                    const float s0 = pr[kb][nt][0] * p.scale, s1 = pr[kb][nt][1] * p.scale, s2 = pr[kb][nt][2] * p.scale,
                                s3 = pr[kb][nt][3] * p.scale;
                    dsa[rb][kb][nt * 2 + 0] = pack_bf16x2(s0 * (dp[kb][nt][0] - d0), s1 * (dp[kb][nt][1] - d0));
                    dsa[rb][kb][nt * 2 + 1] = pack_bf16x2(s2 * (dp[kb][nt][2] - d1), s3 * (dp[kb][nt][3] - d1));
                }
        } else {
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
#pragma unroll
                for (int i = 0; i < 4; ++i) pa[rb][kb][i] = dsa[rb][kb][i] = 0u;
        }
    }

    float acc[(D + 15) / 16 * 2][4];
    // dV (keys kb) = sum over query blocks of P^T dO; V is no longer needed, dV rows take its place
#pragma unroll
    for (int kb = 0; kb < NB; ++kb) {
        if (kb < n_b) {
#pragma unroll
            for (int nt = 0; nt < (D + 15) / 16 * 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int rb = 0; rb < NB; ++rb) {
                if (rb < n_b) {
                    const uint32_t at[4] = {transpose8x8(pa[rb][kb][0]), transpose8x8(pa[rb][kb][2]), transpose8x8(pa[rb][kb][1]),
                                            transpose8x8(pa[rb][kb][3])};
                    fast_into_d<D>(acc, at, lane_row_a(g_s, rb, s, lane, s.zero));
                }
            }
            fast_stage<D>(acc, lane_row_a(v_s, kb, s, lane, s.dump));
        }
    }
    __syncwarp();
    // dQ (queries rb) = sum over key blocks of (scale dS) K; dO is no longer needed, dQ rows take its place
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
        if (rb < n_b) {
#pragma unroll
            for (int nt = 0; nt < (D + 15) / 16 * 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int kb = 0; kb < NB; ++kb)
                if (kb < n_b) fast_into_d<D>(acc, dsa[rb][kb], lane_row_a(k_s, kb, s, lane, s.zero));
            fast_stage<D>(acc, lane_row_a(g_s, rb, s, lane, s.dump));
        }
    }
    __syncwarp();
    // dK (keys kb) = sum over query blocks of (scale dS)^T Q; K is no longer needed, dK rows take its place
#pragma unroll
    for (int kb = 0; kb < NB; ++kb) {
        if (kb < n_b) {
#pragma unroll
            for (int nt = 0; nt < (D + 15) / 16 * 2; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int rb = 0; rb < NB; ++rb) {
                if (rb < n_b) {
                    const uint32_t at[4] = {transpose8x8(dsa[rb][kb][0]), transpose8x8(dsa[rb][kb][2]), transpose8x8(dsa[rb][kb][1]),
                                            transpose8x8(dsa[rb][kb][3])};
                    fast_into_d<D>(acc, at, lane_row_a(q_s, rb, s, lane, s.zero));
                }
            }
            fast_stage<D>(acc, lane_row_a(k_s, kb, s, lane, s.dump));
        }
    }
}

// ---- the pipeline: every warp on its own ---------------------------------------------------------------------
// A warp owns two stages of shared memory, each holding one run (at most 16 * NB rows of q, k, v (, dO, lse)).
// It walks its items (chunk, head) round robin, cuts each item's sequences into runs, and keeps the copies of the
// next run in flight while it computes and stores the current one.  No CTA-wide barrier anywhere: a CTA is just
// as many warps as fit the shared memory.
constexpr uint32_t kSmallHeaderBytes = 1024;     // a row of zeros (512 bytes) and a dump row (512 bytes)
constexpr size_t kSmallSmemBudget = 224 * 1024;  // one CTA per SM

struct StageLayout {
    uint32_t pitch, tile_bytes, lse_off, stage_bytes;
};
__host__ __device__ inline StageLayout stage_layout(int n_tiles, int rows, int head_dim, bool with_lse) {
    StageLayout l;
    // 16 or 32 extra bytes per row make the pitch an odd number of 16-byte units: ldmatrix and stmatrix touch eight
    // rows at one column, which then fall into eight different bank groups
    l.pitch = (uint32_t)head_dim * 2 + ((head_dim / 8) % 2 ? 32 : 16);
    l.tile_bytes = (uint32_t)rows * l.pitch;
    l.lse_off = (uint32_t)n_tiles * l.tile_bytes;
    l.stage_bytes = (l.lse_off + (with_lse ? (uint32_t)rows * 4 : 0) + 127) & ~127u;
    return l;
}

struct Run {
    int a, len, head;       // first token, rows, head
    uint32_t starts;
};

// The sequences of a warp's items, cut into runs.  Lane l holds boundary w0 + l of the current item (a window of
// 32 boundaries): the end of a run is one ballot (the boundaries within 16 * NB rows of its start form a prefix of
// the window; a run also ends where the window does), the starts of its sequences one OR over the lanes.
template <int NB>
struct RunWalker {
    const SmallParams& p;
    int lane, dc, dh;
    int chunk, head;        // current item
    int s0, n_s;            // its sequences [s0, s0 + n_s)
    int next_s0, next_s1;   // the following item's, loaded one item ahead
    int i, w0;              // next sequence to place (relative to s0); first boundary of the window (-1: none loaded)
    int mine, above;        // boundary w0 + lane and w0 + lane + 1

    __device__ __forceinline__ void following(int& c, int& h) const {
        c = chunk + dc;
        h = head + dh;
        if (h >= p.n_heads) {
            h -= p.n_heads;
            ++c;
        }
    }
    __device__ __forceinline__ void prefetch_following() {
        int c, h;
        following(c, h);
        next_s0 = next_s1 = 0;
        if (c < p.n_chunks) {
            next_s0 = p.first_seq[c];
            next_s1 = p.first_seq[c + 1];
        }
    }
    __device__ __forceinline__ RunWalker(const SmallParams& params, int warp_global, int warps_total, int lane_)
        : p(params), lane(lane_), dc(warps_total / params.n_heads), dh(warps_total % params.n_heads),
          chunk(warp_global / params.n_heads), head(warp_global % params.n_heads), s0(0), n_s(0), next_s0(0), next_s1(0),
          i(0), w0(-1), mine(0), above(0) {
        if (chunk < p.n_chunks) {
            s0 = p.first_seq[chunk];
            n_s = p.first_seq[chunk + 1] - s0;
            prefetch_following();
        }
    }
    __device__ __forceinline__ bool next(Run& r) {
        while (chunk < p.n_chunks) {
            if (i >= n_s) {             // the item is exhausted
                following(chunk, head);
                s0 = next_s0;
                n_s = next_s1 - next_s0;
                i = 0;
                w0 = -1;
                if (chunk < p.n_chunks) prefetch_following();
                continue;
            }
            if (w0 < 0 || i >= w0 + 31) {
                w0 = i;
                mine = w0 + lane <= n_s ? p.cu[s0 + w0 + lane] : INT_MAX;
                above = __shfl_down_sync(0xffffffffu, mine, 1);
            }
            const int a = __shfl_sync(0xffffffffu, mine, i - w0);
            int j = w0 + __popc(__ballot_sync(0xffffffffu, mine - a <= 16 * NB)) - 1;
            const bool too_long = j <= i;       // refused by the check kernel; never computed
            if (too_long) j = i + 1;
            const int len = __shfl_sync(0xffffffffu, mine, j - w0) - a;
            const uint32_t bit = (w0 + lane >= i && w0 + lane < j && above > mine) ? 1u << ((mine - a) & 31) : 0u;
            const uint32_t starts = __reduce_or_sync(0xffffffffu, bit);
            i = j;
            if (len > 0 && len <= 16 * NB && !too_long) {
                r.a = a;
                r.len = len;
                r.head = head;
                r.starts = starts;
                return true;
            }
        }
        return false;
    }
};

template <int DT, int N_TILES, bool WITH_LSE>
__device__ __forceinline__ void issue_run(const SmallParams& p, const Run& r, const StageLayout& l, uint32_t stage,
                                          const __nv_bfloat16* const (&src)[N_TILES], int lane) {
    const int c16 = DT ? DT / 8 : p.head_dim / 8;
    const size_t base = (size_t)r.a * (size_t)p.row_stride + (size_t)r.head * p.head_dim;
    if (DT != 0 && 32 % (DT ? DT / 8 : 1) == 0) {
        // a lane keeps its 16-byte column and steps down the rows
        constexpr int kC16 = DT ? DT / 8 : 1, kStep = 32 / kC16;
        const int c = lane % kC16, r0 = lane / kC16;
        size_t off = base + (size_t)r0 * (size_t)p.row_stride + (size_t)c * 8;
        const size_t off_step = (size_t)kStep * (size_t)p.row_stride;
        uint32_t dst = stage + (uint32_t)r0 * l.pitch + (uint32_t)c * 16;
        for (int row = r0; row < r.len; row += kStep, off += off_step, dst += kStep * l.pitch) {
#pragma unroll
            for (int t = 0; t < N_TILES; ++t) copy_async_16(dst + (uint32_t)t * l.tile_bytes, src[t] + off);
        }
    } else {
        for (int idx = lane; idx < r.len * c16; idx += 32) {
            const int row = idx / c16, c = idx - row * c16;
            const size_t off = base + (size_t)row * (size_t)p.row_stride + (size_t)c * 8;
            const uint32_t dst = stage + (uint32_t)row * l.pitch + (uint32_t)c * 16;
#pragma unroll
            for (int t = 0; t < N_TILES; ++t) copy_async_16(dst + (uint32_t)t * l.tile_bytes, src[t] + off);
        }
    }
    if (WITH_LSE && lane < r.len) copy_async_4(stage + l.lse_off + lane * 4, p.lse + (size_t)r.head * p.total_tokens + r.a + lane);
}

template <int DT>
__device__ __forceinline__ void store_run(const SmallParams& p, const Run& r, const StageLayout& l, uint32_t tile, __nv_bfloat16* dst,
                                          int lane) {
    const int c16 = DT ? DT / 8 : p.head_dim / 8;
    dst += (size_t)r.a * (size_t)p.row_stride + (size_t)r.head * p.head_dim;
    if (DT != 0 && 32 % (DT ? DT / 8 : 1) == 0) {
        constexpr int kC16 = DT ? DT / 8 : 1, kStep = 32 / kC16;
        const int c = lane % kC16, r0 = lane / kC16;
        __nv_bfloat16* out = dst + (size_t)r0 * (size_t)p.row_stride + (size_t)c * 8;
        const size_t out_step = (size_t)kStep * (size_t)p.row_stride;
        uint32_t from = tile + (uint32_t)r0 * l.pitch + (uint32_t)c * 16;
        for (int row = r0; row < r.len; row += kStep, out += out_step, from += kStep * l.pitch)
            *reinterpret_cast<uint4*>(out) = ld_shared_16(from);
    } else {
        for (int idx = lane; idx < r.len * c16; idx += 32) {
            const int row = idx / c16, c = idx - row * c16;
            const uint4 val = ld_shared_16(tile + (uint32_t)row * l.pitch + (uint32_t)c * 16);
            *reinterpret_cast<uint4*>(dst + (size_t)row * (size_t)p.row_stride + (size_t)c * 8) = val;
        }
    }
}

// DT = head dimension if known at compile time (every loop unrolled), 0 = read it from the parameters.
template <int DT, int NB, bool BWD>
__global__ void __launch_bounds__(512, 1) small_attn_kernel(const SmallParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int N_TILES = BWD ? 4 : 3;
    if (p.hdr->call_bad) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    const StageLayout l = stage_layout(N_TILES, 16 * NB, DT ? DT : p.head_dim, BWD);
    const uint32_t zero = smem_u32(smem);
    const unsigned two = p.stages == 2 ? 1u : 0u;
    uint8_t* my_gen = smem + kSmallHeaderBytes + (size_t)warp * (size_t)p.stages * l.stage_bytes;
    const uint32_t my_stages = smem_u32(my_gen);
    if (threadIdx.x < 128) reinterpret_cast<uint32_t*>(smem)[threadIdx.x] = 0u;
    __syncthreads();        // the only one: the row of zeros
    const __nv_bfloat16* const src4[4] = {p.q, p.k, p.v, BWD ? p.d_o : p.v};
    const __nv_bfloat16* const src3[3] = {p.q, p.k, p.v};

    RunWalker<NB> walker(p, (int)blockIdx.x * n_warps + warp, (int)gridDim.x * n_warps, lane);
    Run cur, nxt;
    if (!walker.next(cur)) return;
    if (BWD) issue_run<DT, 4, true>(p, cur, l, my_stages, src4, lane); else issue_run<DT, 3, false>(p, cur, l, my_stages, src3, lane);
    copy_async_commit();
    for (unsigned it = 0;; ++it) {
        const uint32_t st = my_stages + (it & two) * l.stage_bytes, st_nxt = my_stages + ((it + 1) & two) * l.stage_bytes;
        const bool more = walker.next(nxt);
        if (two) {
            if (more) {
                if (BWD) issue_run<DT, 4, true>(p, nxt, l, st_nxt, src4, lane); else issue_run<DT, 3, false>(p, nxt, l, st_nxt, src3, lane);
            }
            copy_async_commit();
            copy_async_wait<1>();       // everything but the group just committed: this run's rows are here
        } else {
            copy_async_wait<0>();
        }
        __syncwarp();

        const SeqView sv{zero, zero + 512, l.pitch, cur.len, cur.starts};
        const float* lse_s = reinterpret_cast<const float*>(my_gen + (size_t)(it & two) * l.stage_bytes + l.lse_off);
        float* lse_out = p.lse + (size_t)cur.head * p.total_tokens + cur.a;
        if (BWD) {
            if (DT != 0)
                bwd_sequence_fast<DT ? DT : 16, NB>(p, sv, st, st + l.tile_bytes, st + 2 * l.tile_bytes, st + 3 * l.tile_bytes, lse_s, lane);
            else
                bwd_sequence<NB>(p, sv, st, st + l.tile_bytes, st + 2 * l.tile_bytes, st + 3 * l.tile_bytes, lse_s, lane);
            __syncwarp();
            store_run<DT>(p, cur, l, st + 3 * l.tile_bytes, p.dq, lane);
            store_run<DT>(p, cur, l, st + l.tile_bytes, p.dk, lane);
            store_run<DT>(p, cur, l, st + 2 * l.tile_bytes, p.dv, lane);
        } else {
            if (DT != 0)
                fwd_sequence_fast<DT ? DT : 16, NB>(p, sv, st, st + l.tile_bytes, st + 2 * l.tile_bytes, lse_out, lane);
            else
                fwd_sequence<NB>(p, sv, st, st + l.tile_bytes, st + 2 * l.tile_bytes, lse_out, lane);
            __syncwarp();
            store_run<DT>(p, cur, l, st, p.o, lane);
        }
        __syncwarp();                   // the stage is free for the copies issued in the next iteration
        if (!more) break;
        cur = nxt;
        if (!two) {                     // one stage: the next run's copies start now, other warps compute meanwhile
            if (BWD) issue_run<DT, 4, true>(p, cur, l, st, src4, lane); else issue_run<DT, 3, false>(p, cur, l, st, src3, lane);
            copy_async_commit();
        }
    }
    copy_async_wait<0>();
}

// First kernel of a call on the short-sequence path: the boundaries must start at 0, end at total_tokens,
// never decrease, and no sequence may exceed the declared maximum; otherwise the status word says so and the
// attention kernel computes nothing.  Then first_seq[c] = first sequence that starts at or after position
// c * chunk, for c = 0 .. n_chunks.  `which` = 0 forward, 1 backward: no CTA time spans are recorded here.
__global__ void __launch_bounds__(1024) small_check_kernel(const int32_t* __restrict__ cu, int32_t n_seqs, int32_t total_tokens,
                                                           int32_t max_len, int32_t chunk, int32_t n_chunks, int32_t* first_seq,
                                                           WorkspaceHeader* hdr, int which) {
    int bad = (threadIdx.x == 0 && (cu[0] != 0 || cu[n_seqs] != total_tokens)) ? 1 : 0;
    for (int i = threadIdx.x; i < n_seqs; i += 1024) {
        const int32_t len = cu[i + 1] - cu[i];
        bad |= (len < 0 || len > max_len) ? 1 : 0;
    }
    bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        header_begin_call(hdr, bad != 0);
        hdr->n_ctas[which] = 0;
    }
    if (bad) return;
    for (int i = threadIdx.x; i <= n_seqs; i += 1024) {
        const int32_t here = cu[i], before = i > 0 ? cu[i - 1] : -1;
        const int c_hi = min(here / chunk, n_chunks);
        for (int c = before < 0 ? 0 : before / chunk + 1; c <= c_hi; ++c) first_seq[c] = i;
    }
    if (threadIdx.x == 0)
        for (int c = total_tokens / chunk + 1; c <= n_chunks; ++c) first_seq[c] = n_seqs;
}

// Token positions per chunk: 64, less for small batches so that every warp of the grid still gets a few items
// (at least 16: the scratch for first_seq is sized for that).
int pick_chunk(int32_t total_tokens, int32_t n_heads, int n_sms) {
    int chunk = 64;
    while (chunk > 16 && (long long)((total_tokens + chunk - 1) / chunk) * n_heads < 4LL * n_sms * 8) chunk /= 2;
    return chunk;
}

// Warps per CTA: as many pairs of stages as fit the shared memory of an SM, at most 16.
int pick_warps(int n_tiles, int rows, int head_dim, bool with_lse, int stages) {
    const size_t per_warp = (size_t)stages * (size_t)stage_layout(n_tiles, rows, head_dim, with_lse).stage_bytes;
    const int warps = (int)((kSmallSmemBudget - kSmallHeaderBytes) / per_warp);
    return warps > 16 ? 16 : warps < 1 ? 1 : warps;
}

}  // namespace

bool small_path_fits(int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen) {
    // first_seq has 2 n_seqs + 1 slots (the work list's order and prefix arrays) and chunks have at least 16
    // positions: enough whenever the declared sizes agree with each other
    return max_seqlen <= kSmallSeqMaxLen && (int64_t)total_tokens <= (int64_t)n_seqs * max_seqlen;
}

cudaError_t launch_small_check(bool backward, const int32_t* cu_seqlens, int32_t n_seqs, int32_t total_tokens, int32_t max_seqlen,
                               int32_t n_heads, WorkspaceHeader* hdr, int32_t* first_seq, int n_sms, cudaStream_t stream) {
    const int chunk = pick_chunk(total_tokens, n_heads, n_sms);
    small_check_kernel<<<1, 1024, 0, stream>>>(cu_seqlens, n_seqs, total_tokens, max_seqlen, chunk, (total_tokens + chunk - 1) / chunk,
                                               first_seq, hdr, backward ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_small_attn(bool backward, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* d_o, float* lse, const int32_t* cu_seqlens, int32_t total_tokens,
                              int32_t max_seqlen, int32_t n_heads, int32_t head_dim, int64_t row_stride, bool causal, float scale,
                              __nv_bfloat16* o, __nv_bfloat16* dq, __nv_bfloat16* dk, __nv_bfloat16* dv, WorkspaceHeader* hdr,
                              const int32_t* first_seq, int n_sms, cudaStream_t stream) {
    const int n_tiles = backward ? 4 : 3;
    SmallParams p{};
    p.q = q;
    p.k = k;
    p.v = v;
    p.d_o = d_o;
    p.o = o;
    p.dq = dq;
    p.dk = dk;
    p.dv = dv;
    p.lse = lse;
    p.cu = cu_seqlens;
    p.first_seq = first_seq;
    p.hdr = hdr;
    p.n_heads = n_heads;
    p.head_dim = head_dim;
    p.total_tokens = total_tokens;
    p.chunk = pick_chunk(total_tokens, n_heads, n_sms);
    p.n_chunks = (total_tokens + p.chunk - 1) / p.chunk;
    p.causal = causal ? 1 : 0;
    p.row_stride = row_stride;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    const int rows = max_seqlen <= 16 ? 16 : 32;
    // Runs of up to 32 rows: a stage is twice as large and a pass four times as long, so more warps per SM (one stage
    // each, the other warps' arithmetic hiding a warp's copies) beat fewer warps with two stages (32 tokens per sequence,
    // forward + backward: 1.49 -> 1.21 ms).  Runs of up to 16 rows: two stages are slightly ahead (1.06 vs 1.07 ms).
    p.stages = rows == 32 ? 1 : 2;
    const int warps = pick_warps(n_tiles, rows, head_dim, backward, p.stages);
    const size_t smem = kSmallHeaderBytes + (size_t)warps * p.stages * stage_layout(n_tiles, rows, head_dim, backward).stage_bytes;
    const long long n_items = (long long)p.n_chunks * n_heads;
    const unsigned grid = (unsigned)(n_items < (long long)n_sms * warps ? (n_items + warps - 1) / warps : n_sms);
    auto launch = [&](auto kern) {
        cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        kern<<<grid, 32 * warps, smem, stream>>>(p);
        return cudaGetLastError();
    };
    const bool one = max_seqlen <= 16;
#define DCP_SMALL_DISPATCH(DT)                                                                                      \
    return backward ? (one ? launch(small_attn_kernel<DT, 1, true>) : launch(small_attn_kernel<DT, 2, true>))      \
                    : (one ? launch(small_attn_kernel<DT, 1, false>) : launch(small_attn_kernel<DT, 2, false>))
    if (head_dim == 128) { DCP_SMALL_DISPATCH(128); }
    if (head_dim == 64) { DCP_SMALL_DISPATCH(64); }
    if (head_dim == 72) { DCP_SMALL_DISPATCH(72); }      // the paper's 2-D model (Section 4.1)
    DCP_SMALL_DISPATCH(0);
#undef DCP_SMALL_DISPATCH
}

}  // namespace dcp
