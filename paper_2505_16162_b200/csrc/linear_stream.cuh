// Weight-streaming linear kernel for bf16 weights and up to 8 activation rows (sm_100a).
//
// One persistent CTA per SM.  A producer warp streams the CTA's share of the weight matrix through a
// shared-memory ring with bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts), one
// 2 KB row segment per copy, and streams the matching slices of the activations through a second, small
// ring.  Eight consumer warps turn each 16-row x 1024-column weight tile into tensor-core work:
// ldmatrix for the weight fragments, mma.sync m16n8k16 with the weights as the 16-row operand and the
// (at most 8) activation rows as the 8-column operand.  Activations are fp32; each value is split into
// three bf16 terms (hi + mid + lo, 24 mantissa bits together) and multiplied separately, so products are
// exact and the result has fp32-accumulate accuracy.  The contraction is HBM-bound: the tensor pipe is
// used because it makes the per-byte instruction cost independent of the number of rows, not for FLOPs.
//
// Work split: the CTA owns a contiguous range of output units (balanced to +-1 across CTAs), cut into
// groups of at most 16 rows (8 gate + 8 up rows for the SwiGLU pair), processed in batches of up to 8
// groups.  Inside a batch the loop runs over column tiles (outer) and groups (inner), so an activation
// slice is staged and split once per column tile.  The 8 consumer warps each own a 128-column slot of
// every tile; their partial sums meet in shared memory in warp order at the end of a batch.  The sum
// order of an output therefore depends only on K, never on the row count M or on the grid.
//
// Every wait on an mbarrier is bounded: after SPIN_LIMIT polls the thread raises a CTA-wide abort flag,
// records a code in *err, and all threads fall through to the end of the kernel without further waits.
#pragma once
#include "kernels.cuh"

namespace knnssd {
namespace stream {

constexpr int SEG = 1024;                    // bf16 columns per tile
constexpr int WROWS = 16;                    // rows per weight tile (one mma M)
constexpr int WPITCH = SEG * 2 + 16;         // bytes; (pitch / 16) odd -> ldmatrix rows hit distinct banks
constexpr int WSTAGE = WROWS * WPITCH;
constexpr int XPITCH = SEG * 4 + 32;         // bytes; token rows 32 B apart modulo 128 -> conflict-free float2 reads
constexpr int NCW = 8;                       // consumer warps
constexpr int SLOT = SEG / NCW;              // columns per consumer warp per tile (128 = 8 k16 steps)
constexpr int KSTEPS = SLOT / 16;
constexpr int GB = 8;                        // groups per batch
constexpr int NTHREADS = (NCW + 1) * 32;
constexpr int RED_BYTES = NCW * GB * 32 * 4 * 4;
constexpr int SS_BYTES = NCW * 8 * 4;
constexpr int MAX_SMEM = 232448;             // 227 KB
constexpr unsigned SPIN_LIMIT = 20000000u;

__host__ __device__ constexpr int xstage_bytes(int MT) { return (MT + 1) * XPITCH; }   // M token rows + the gain row
__host__ __device__ constexpr int n_wstages(int MT) {
    return (MAX_SMEM - 2 * xstage_bytes(MT) - RED_BYTES - SS_BYTES - 1024) / WSTAGE;
}
__host__ __device__ constexpr int smem_bytes(int MT) {
    return n_wstages(MT) * WSTAGE + 2 * xstage_bytes(MT) + RED_BYTES + SS_BYTES + 1024;
}

struct Args {
    const bf16_t *W[3];
    int rows[3];
    int units;          // outputs (SWIGLU: d_ff, each unit = one gate row + one up row)
    int K;              // n_in, multiple of 128
    const float *x;     // [M][K]
    const float *gain;  // [K] or nullptr
    float eps;
    float *y;           // [M][units]
    int epi;
    int M;              // 1..8
    int *err;           // device int: set non-zero if a bounded wait gave up
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the barrier never flipped.
__device__ __forceinline__ bool mbar_wait(uint64_t *b, uint32_t parity, volatile int *abort_flag, int *err, int code) {
    unsigned spins = 0;
    while (!mbar_try_wait(b, parity)) {
        if (*abort_flag) return false;
        if (++spins > SPIN_LIMIT) {
            *abort_flag = 1;
            atomicExch(err, code);
            return false;
        }
    }
    return true;
}
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *b) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(b))
                 : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &a0, uint32_t &a1, uint32_t &a2, uint32_t &a3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// v = hi + mid + lo with each term a bf16 (round to nearest even); residuals are exact in fp32.
__device__ __forceinline__ void split3(float v, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
    hi = float_to_bf16_rne(v);
    const float r1 = v - __uint_as_float(hi << 16);
    mid = float_to_bf16_rne(r1);
    const float r2 = r1 - __uint_as_float(mid << 16);
    lo = float_to_bf16_rne(r2);
}

// Even split of n items into parts: part p covers [lo, hi).
__device__ __forceinline__ void even_part(int n, int parts, int p, int &lo, int &hi) {
    lo = (int)(((long long)n * p) / parts);
    hi = (int)(((long long)n * (p + 1)) / parts);
}

template <int MT>
__global__ void __launch_bounds__(NTHREADS, 1) linear_stream_kernel(const Args a) {
    constexpr int WS = n_wstages(MT);
    constexpr int XST = xstage_bytes(MT);
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *wring = smem;
    unsigned char *xring = smem + WS * WSTAGE;
    float *red = reinterpret_cast<float *>(xring + 2 * XST);
    float *red_ss = red + RED_BYTES / 4;
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(red_ss) + SS_BYTES);
    uint64_t *full_w = bars, *empty_w = bars + WS, *full_x = bars + 2 * WS, *empty_x = bars + 2 * WS + 2;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * WS + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < WS; ++s) { mbar_init(&full_w[s], 1); mbar_init(&empty_w[s], NCW); }
        for (int s = 0; s < 2; ++s) { mbar_init(&full_x[s], 1); mbar_init(&empty_x[s], NCW); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const bool swiglu = a.epi == EPI_SWIGLU;
    const int gsz = swiglu ? 8 : 16;                       // units per group
    int u_lo, u_hi;
    even_part(a.units, gridDim.x, blockIdx.x, u_lo, u_hi);
    const int n_units = u_hi - u_lo;
    const int n_groups = (n_units + gsz - 1) / gsz;
    const int n_batches = (n_groups + GB - 1) / GB;
    const int n_kt = (a.K + SEG - 1) / SEG;
    const bool normed = a.gain != nullptr;

    if (warp == NCW) {
        // ------------------------------ producer ------------------------------
        int w_use = 0, x_use = 0;
        bool alive = true;
        for (int b = 0; b < n_batches && alive; ++b) {
            const int g0 = b * GB, g1 = min(n_groups, g0 + GB);
            for (int kt = 0; kt < n_kt && alive; ++kt) {
                const int c0 = kt * SEG, segc = min(SEG, a.K - c0);
                {   // activation slice (+ gain slice)
                    const int xs = x_use & 1, it = x_use >> 1;
                    if (it > 0) alive = mbar_wait(&empty_x[xs], (it - 1) & 1, abort_flag, a.err, 2);
                    if (!alive) break;
                    if (lane == 0) mbar_expect_tx(&full_x[xs], (uint32_t)(a.M + (normed ? 1 : 0)) * segc * 4);
                    __syncwarp();
                    unsigned char *dst = xring + xs * XST;
                    if (lane < a.M) bulk_g2s(dst + lane * XPITCH, a.x + (size_t)lane * a.K + c0, segc * 4, &full_x[xs]);
                    if (lane == MT && normed) bulk_g2s(dst + MT * XPITCH, a.gain + c0, segc * 4, &full_x[xs]);
                    ++x_use;
                }
                for (int g = g0; g < g1 && alive; ++g) {
                    int lo, hi;
                    even_part(n_units, n_groups, g, lo, hi);
                    const int nu = hi - lo;                  // units in this group (<= gsz)
                    const int ws = w_use % WS, it = w_use / WS;
                    if (it > 0) alive = mbar_wait(&empty_w[ws], (it - 1) & 1, abort_flag, a.err, 3);
                    if (!alive) break;
                    if (lane == 0) mbar_expect_tx(&full_w[ws], (uint32_t)(swiglu ? 2 * nu : nu) * segc * 2);
                    __syncwarp();
                    if (lane < WROWS) {
                        const int r = swiglu ? (lane & 7) : lane;
                        if (r < nu) {
                            int u = u_lo + lo + r;
                            const bf16_t *src;
                            if (swiglu) {
                                src = a.W[lane >> 3] + (size_t)u * a.K;
                            } else {
                                int which = 0;
                                if (u >= a.rows[0]) { u -= a.rows[0]; which = 1; }
                                if (which == 1 && u >= a.rows[1]) { u -= a.rows[1]; which = 2; }
                                src = a.W[which] + (size_t)u * a.K;
                            }
                            bulk_g2s(wring + ws * WSTAGE + lane * WPITCH, src + c0, segc * 2, &full_w[ws]);
                        }
                    }
                    ++w_use;
                }
            }
        }
        if (!alive) {   // give copies already in flight time to land before the CTA's shared memory goes away
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        }
    } else {
        // ------------------------------ consumers ------------------------------
        const int g8 = lane >> 2, t4 = lane & 3;
        const int lm_row = (lane & 7) + ((lane >> 3) & 1) * 8, lm_col = (lane >> 4) * 8;   // ldmatrix source of this lane
        int w_use = 0, x_use = 0;
        bool alive = true;
        for (int b = 0; b < n_batches; ++b) {
            const int g0 = b * GB, g1 = min(n_groups, g0 + GB);
            float acc[GB][4];
#pragma unroll
            for (int i = 0; i < GB; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
            float ss = 0.f;
            for (int kt = 0; kt < n_kt; ++kt) {
                const int c0 = kt * SEG, segc = min(SEG, a.K - c0);
                const bool slot_valid = warp * SLOT < segc;
                uint32_t bh[KSTEPS][2], bm[KSTEPS][2], bl[KSTEPS][2];
                {
                    const int xs = x_use & 1, it = x_use >> 1;
                    if (alive) alive = mbar_wait(&full_x[xs], it & 1, abort_flag, a.err, 4);
                    const unsigned char *xst = xring + xs * XST;
#pragma unroll
                    for (int j = 0; j < KSTEPS; ++j) {
                        float v[4] = {0.f, 0.f, 0.f, 0.f};
                        if (alive && slot_valid && g8 < a.M) {
                            const int col = warp * SLOT + j * 16 + 2 * t4;
                            const float2 p0 = *reinterpret_cast<const float2 *>(xst + g8 * XPITCH + col * 4);
                            const float2 p1 = *reinterpret_cast<const float2 *>(xst + g8 * XPITCH + (col + 8) * 4);
                            v[0] = p0.x; v[1] = p0.y; v[2] = p1.x; v[3] = p1.y;
                            if (normed) {
                                ss = fmaf(v[0], v[0], ss); ss = fmaf(v[1], v[1], ss);
                                ss = fmaf(v[2], v[2], ss); ss = fmaf(v[3], v[3], ss);
                                const float2 q0 = *reinterpret_cast<const float2 *>(xst + MT * XPITCH + col * 4);
                                const float2 q1 = *reinterpret_cast<const float2 *>(xst + MT * XPITCH + (col + 8) * 4);
                                v[0] *= q0.x; v[1] *= q0.y; v[2] *= q1.x; v[3] *= q1.y;
                            }
                        }
                        uint32_t h[4], m[4], l[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) split3(v[e], h[e], m[e], l[e]);
                        bh[j][0] = h[0] | (h[1] << 16); bh[j][1] = h[2] | (h[3] << 16);
                        bm[j][0] = m[0] | (m[1] << 16); bm[j][1] = m[2] | (m[3] << 16);
                        bl[j][0] = l[0] | (l[1] << 16); bl[j][1] = l[2] | (l[3] << 16);
                    }
                    __syncwarp();
                    if (alive && lane == 0) mbar_arrive(&empty_x[xs]);
                    ++x_use;
                }
#pragma unroll
                for (int gi = 0; gi < GB; ++gi) {
                    if (g0 + gi >= g1) break;
                    const int ws = w_use % WS, it = w_use / WS;
                    if (alive) alive = mbar_wait(&full_w[ws], it & 1, abort_flag, a.err, 5);
                    if (alive && slot_valid) {
                        const uint32_t base = smem_u32(wring + ws * WSTAGE) + lm_row * WPITCH + (warp * SLOT + lm_col) * 2;
#pragma unroll
                        for (int j = 0; j < KSTEPS; ++j) {
                            uint32_t a0, a1, a2, a3;
                            ldmatrix_x4(base + j * 32, a0, a1, a2, a3);
                            mma_bf16(acc[gi], a0, a1, a2, a3, bl[j][0], bl[j][1]);
                            mma_bf16(acc[gi], a0, a1, a2, a3, bm[j][0], bm[j][1]);
                            mma_bf16(acc[gi], a0, a1, a2, a3, bh[j][0], bh[j][1]);
                        }
                    }
                    __syncwarp();
                    if (alive && lane == 0) mbar_arrive(&empty_w[ws]);
                    ++w_use;
                }
            }
            // ---- batch end: partial sums of the 8 column slots meet in shared memory, in warp order ----
#pragma unroll
            for (int gi = 0; gi < GB; ++gi)
                *reinterpret_cast<float4 *>(red + ((warp * GB + gi) * 32 + lane) * 4) =
                    make_float4(acc[gi][0], acc[gi][1], acc[gi][2], acc[gi][3]);
            if (normed) {
                ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                if (t4 == 0) red_ss[warp * 8 + g8] = ss;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
            if (alive) {
                const int ng = g1 - g0;
                const int per_group = gsz * 8;                        // (unit, token) pairs per group
                for (int idx = tid; idx < ng * per_group; idx += NCW * 32) {
                    const int gi = idx / per_group, rem = idx % per_group;
                    const int r = rem >> 3, n = rem & 7;              // unit within group, token
                    int lo, hi;
                    even_part(n_units, n_groups, g0 + gi, lo, hi);
                    if (r >= hi - lo || n >= a.M) continue;
                    const int src_lane = r * 4 + (n >> 1), reg = n & 1;  // rows 0..7 of the tile: regs 0,1; rows 8..15: regs 2,3
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int w = 0; w < NCW; ++w) {
                        const float *p = red + ((w * GB + gi) * 32 + (swiglu ? src_lane : ((r & 7) * 4 + (n >> 1)))) * 4;
                        if (swiglu) { s0 += p[reg]; s1 += p[2 + reg]; }
                        else s0 += p[(r >> 3) * 2 + reg];
                    }
                    float ri = 1.0f;
                    if (normed) {
                        float tot = 0.f;
#pragma unroll
                        for (int w = 0; w < NCW; ++w) tot += red_ss[w * 8 + n];
                        ri = 1.0f / sqrtf(tot / (float)a.K + a.eps);
                    }
                    float *yp = a.y + (size_t)n * a.units + (u_lo + lo + r);
                    if (swiglu) {
                        const float gt = s0 * ri, up = s1 * ri;
                        *yp = gt / (1.0f + expf(-gt)) * up;
                    } else if (a.epi == EPI_ADD) {
                        *yp += s0 * ri;
                    } else {
                        *yp = s0 * ri;
                    }
                }
            }
            asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
        }
    }
}

}  // namespace stream
}  // namespace knnssd
