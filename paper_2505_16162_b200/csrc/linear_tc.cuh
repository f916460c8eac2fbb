// Weight-streaming linear map for up to 16 rows on the 5th-generation tensor cores (stand-alone; the passes do not use
// it yet).  y[m][u] = sum_i W[u][i] x[m][i], W bf16 [n_out][K], x fp32 given as two bf16 terms (hi + lo).
//
// The decode passes (Sec. 4.2: k draft steps of one row, one verification pass of k + 1 rows) are bound by the HBM
// traffic of the weights; on mma.sync their cost grows with the rows beyond 8 (twice the MMAs per weight tile).  Here
// the weights are the 128-row operand of tcgen05.mma and the pass's rows its 16 columns: M = 128 units, N = 16 rows,
// K = 16 per instruction, accumulator 128 lanes x 16 columns of tensor memory, so any row count up to 16 costs the
// same.  A CTA takes one work item = (tile of 128 units, chunk of the input columns); the chunks' partial sums are
// written out and added in chunk order by a second kernel (fixed order: the result does not depend on timing).
// Operands come through TMA (128-byte swizzle) into a ring of 5 stages of 20 KB (16 KB of weights, 2 x 2 KB of x);
// two CTAs share an SM.
// All waits are bounded.
#pragma once

#include "prefill.cuh"

namespace knnssd {
namespace lintc {

using prefill::pf_wait;
using prefill::tma_load_2d;
using prefill::umma_bf16;
using prefill::umma_commit;
using prefill::umma_desc;
using prefill::umma_idesc;
using stream::mbar_init;
using stream::smem_u32;

constexpr int TM = 128;                     // units per tile (accumulator lanes)
constexpr int TN = 16;                      // rows of x (accumulator columns)
constexpr int BK = 64;                      // input columns per stage
constexpr int STAGES = 5;                     // 5 x 20 KB: two CTAs per SM, one streams while the other starts or drains
constexpr int W_BYTES = TM * BK * 2;        // 16 KB
constexpr int X_BYTES = TN * BK * 2;        // 2 KB per term
constexpr int STAGE_BYTES = W_BYTES + 2 * X_BYTES;
constexpr int THREADS = 192;                // warp 0: TMA; warp 1: MMA issue + tensor-memory owner; warps 2..5: epilogue
constexpr int SMEM = STAGES * STAGE_BYTES + 1024 + 256;
constexpr int TMEM_COLS = 32;               // smallest allocation; 16 columns are used

struct Args {
    int M;          // live rows (1..16)
    int K;          // input width, a multiple of BK
    int n_out;
    int kc;         // chunks of the input columns
    int kb_per;     // k-blocks (of BK columns) per chunk
    float *part;    // [kc][M][n_out] partial sums
    int *err;
};

// tw: weights [n_out][K], boxes of 128 rows x 64 columns; tx: x planes [32][K] (rows 0..15 hi, 16..31 lo), boxes of
// 16 rows x 64 columns.  grid = (ceil(n_out / 128), kc).
__global__ void __launch_bounds__(THREADS, 2)
linear_tc_kernel(const __grid_constant__ CUtensorMap tw, const __grid_constant__ CUtensorMap tx, Args g) {
    extern __shared__ unsigned char lt_smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(lt_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
    volatile int *cta_abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int u0 = blockIdx.x * TM;
    const int kb0 = blockIdx.y * g.kb_per;
    const int nkb = min(g.kb_per, g.K / BK - kb0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1);
        *cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    prefill::tc_fence_before();
    __syncthreads();
    prefill::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int armed = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                if (!pf_wait(&empty[s], ph ^ 1u, cta_abort, g.err, 41)) break;
                unsigned char *st = smem + s * STAGE_BYTES;
                stream::mbar_expect_tx(&full[s], STAGE_BYTES);
                tma_load_2d(st, &tw, (kb0 + kb) * BK, u0, &full[s]);
                tma_load_2d(st + W_BYTES, &tx, (kb0 + kb) * BK, 0, &full[s]);
                tma_load_2d(st + W_BYTES + X_BYTES, &tx, (kb0 + kb) * BK, TN, &full[s]);
                armed = kb + 1;
            }
            if (*cta_abort) {
                for (int kb = (armed > STAGES ? armed - STAGES : 0); kb < armed; ++kb) {
                    unsigned spins = 0;
                    while (!stream::mbar_try_wait(&full[kb % STAGES], (uint32_t)(kb / STAGES) & 1u) && ++spins < prefill::WAIT_LIMIT) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(TN);
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                if (!pf_wait(&full[s], ph, cta_abort, g.err, 42)) break;
                prefill::tc_fence_after();
                const uint32_t w = smem_u32(smem + s * STAGE_BYTES), xh = w + W_BYTES, xl = xh + X_BYTES;
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    const uint64_t dw = umma_desc(w + 32 * k);
                    umma_bf16(tmem, dw, umma_desc(xl + 32 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_bf16(tmem, dw, umma_desc(xh + 32 * k), idesc, 1u);
                }
                umma_commit(&empty[s]);
            }
            umma_commit(acc_full);
        }
    } else {
        const bool ok = __all_sync(0xffffffffu, pf_wait(acc_full, 0u, cta_abort, g.err, 43) && !*cta_abort);
        prefill::tc_fence_after();
        const int q = warp & 3;
        const int u = u0 + 32 * q + lane;
        if (ok) {
            uint32_t r[16];
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                  "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                : "r"(tmem + ((uint32_t)(32 * q) << 16))
                : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (u < g.n_out) {
                float *dst = g.part + (size_t)blockIdx.y * g.M * g.n_out + u;
#pragma unroll
                for (int m = 0; m < TN; ++m)
                    if (m < g.M) dst[(size_t)m * g.n_out] = __uint_as_float(r[m]);
            }
        }
    }
    prefill::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        prefill::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// y[m][u] = sum over chunks, in chunk order, of part[c][m][u].  One thread per output.
__global__ void reduce_chunks_kernel(const float *__restrict__ part, int kc, size_t n, float *__restrict__ y) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int c = 0; c < kc; ++c) s += part[(size_t)c * n + i];
    y[i] = s;
}

// The two bf16 terms of x rows [M][K] into planes [32][K] (rows M..15 and 16 + M..31 stay zero).  grid = M.
__global__ void split_x_kernel(const float *__restrict__ x, int K, bf16_t *__restrict__ planes) {
    const size_t base = (size_t)blockIdx.x * K;
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
        const float v = x[base + i];
        const uint32_t h = float_to_bf16_rne(v);
        planes[base + i] = (bf16_t)h;
        planes[(size_t)TN * K + base + i] = float_to_bf16_rne(v - __uint_as_float(h << 16));
    }
}

}  // namespace lintc
}  // namespace knnssd
