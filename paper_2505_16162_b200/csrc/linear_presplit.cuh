// Consumer half of the weight-streaming linear engine for PRE-SPLIT activations (persistent pass kernel).
//
// Same ring, same tiles, same sum order per output as consume_linear, but the activation operand arrives already
// split into its bf16 terms and laid out fragment by fragment (LinPhase::xs), written once by whoever produced the
// activation.  The consumer therefore spends no arithmetic on the split that every CTA would otherwise repeat:
// per column tile a lane loads four 16-byte pieces per term and row block, one tile ahead of the tensor-core work.
// RMSNorm's scalar comes from per-CTA partial sums of squares that the producer of the row left in LinPhase::ss_in.
//
// NB = row blocks of eight: 1 for passes of up to 8 rows, 2 for 9..16 rows (the second block is a second 8-column
// operand for the same weight fragments; every row is computed exactly as it would be in a one-row pass).
//
// NP > 0 (the paired form; NP = 1: passes of up to 4 rows - every draft step; NP = 3: passes of 9..12 rows): the rows
// are taken four at a time and the two bf16 terms of a row sit in neighbouring columns of ONE 8-column operand
// (column 2 r = hi term of row 4 b + r, 2 r + 1 = its lo term), so a weight fragment takes one MMA per four rows
// instead of two per eight: 1 instead of 2 for up to 4 rows, 3 instead of 4 for 9..12.  A consumer that is faster
// than the HBM stream drains the ring after a barrier and lets the producer run ahead again.  An output is
// still (sum of the lo products) + (sum of the hi products), each sum accumulated over the same k-steps in the same
// order as in the unpaired form: the numbers do not depend on which form computed them.
//
// The epilogue writes what the NEXT map needs: the fp32 result where something reads it as fp32 (projection buffer,
// residual stream, logits) and, for the residual update and the SwiGLU product, the pre-split form (times the next
// RMSNorm's gain) plus this CTA's partial sums of squares.
#pragma once
#include "linear_stream.cuh"

namespace knnssd {
namespace stream {

__device__ __forceinline__ uint4 ld_frag4(const uint32_t *p) { return __ldcg(reinterpret_cast<const uint4 *>(p)); }

// Column groups (of 16 units) a batch of the consumer takes, by kernel form; LinPhase::gb carries it to the producer.
template <int NB, int NP> __host__ __device__ constexpr int groups_per_batch() { return NP == 3 ? GB : GB / NB; }

template <int NB, int NP>
__device__ __forceinline__ void consume_linear_pre(const LinPhase &p, const Ring &r, int cta, int n_cta, int warp, int lane,
                                                   int &w_use, bool &alive) {
    constexpr bool PAIRED = NP > 0;
    static_assert(NP * 4 <= NB * 8, "paired blocks of four rows cover at most the pass's rows");
    constexpr int NX = PAIRED ? NP : NB;                    // operand blocks: of 4 rows (paired) or of 8 rows
    constexpr int NTM = PAIRED ? 1 : NTERM;                 // operand sets (MMAs) per weight fragment and operand block
    // groups per batch: the tile loop is unrolled over them and has to stay small (instruction cache), so two row
    // blocks of eight take half as many groups; the producer is told the same number through LinPhase::gb.  The
    // activation fragments of a column tile are fetched from L2 once per batch, so the 9..12-row form keeps four
    // groups: at two it would pull 0.75 bytes of activations per byte of weights.
    constexpr int GBN = groups_per_batch<NB, NP>();
    constexpr int RW = PAIRED ? 2 : 4;                      // floats a lane leaves per (warp, group, block) for the batch-end sums
    const Share s = make_share(p, cta, n_cta);
    const int tid = warp * 32 + lane;
    const int g8 = lane >> 2, t4 = lane & 3;
    const int lm_row = (lane & 7) + ((lane >> 3) & 1) * 8, lm_col = (lane >> 4) * 8;   // ldmatrix source of this lane
    const bool normed = p.ss_in != nullptr;
    const int nslots = p.K >> 7;
    // this lane's 16-byte pieces: row nb*8 + g8, lane group t4; + slot * SLOT_WORDS + term * 64 + piece * 16
    const uint32_t *xsrow[NX];
    bool row_live[NX];
#pragma unroll
    for (int nb = 0; nb < NX; ++nb) {
        // this lane's operand column: row nb * 8 + g8, both terms; PAIRED: term g8 & 1 of row nb * 4 + g8 / 2
        const int row = PAIRED ? nb * 4 + (g8 >> 1) : nb * 8 + g8;
        row_live[nb] = row < p.M;
        xsrow[nb] = p.xs + (size_t)min(row, p.M - 1) * nslots * SLOT_WORDS + (PAIRED ? (g8 & 1) * 64 : 0) + t4 * 4;
    }
    int ws = w_use % WS, it = w_use / WS;
    float *red = r.red, *red_ss = r.red_ss;

    float ss_acc[NB];                                       // lane 0 of warp w: this CTA's sum of squares of y rows w, w + 8
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) ss_acc[nb] = 0.f;

    for (int b = 0; b < s.n_batches; ++b) {
        const int g0 = b * GBN, ng = min(s.n_groups - g0, GBN);
        float acc[GBN][NX][4];
#pragma unroll
        for (int i = 0; i < GBN; ++i)
#pragma unroll
            for (int nb = 0; nb < NX; ++nb) { acc[i][nb][0] = acc[i][nb][1] = acc[i][nb][2] = acc[i][nb][3] = 0.f; }
        uint4 nx[NX][NTM][4];                                // fragments of the next column tile, block by block, term by term
        auto fetch = [&](int kt) {
            const int slot = kt * NCW + warp;
#pragma unroll
            for (int nb = 0; nb < NX; ++nb) {
                const bool ld = alive && row_live[nb] && slot < nslots;
#pragma unroll
                for (int t = 0; t < NTM; ++t)
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        nx[nb][t][q] = ld ? ld_frag4(xsrow[nb] + (size_t)slot * SLOT_WORDS + t * 64 + q * 16) : make_uint4(0u, 0u, 0u, 0u);
            }
        };
        fetch(0);
        if (b == 0 && normed) {
            // RMSNorm scalar of rows `warp` (and warp + 8) from the producers' partial sums (lanes take CTAs lane,
            // lane + 32, ...); issued after the first fragment fetch so that both round trips to L2 overlap
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                const int row = nb * 8 + warp;
                if (row < p.M) {
                    float tot = 0.f;
                    for (int c = lane; c < n_cta; c += 32) tot += __ldcg(p.ss_in + (size_t)row * n_cta + c);
                    tot = warp_sum(tot);
                    if (lane == 0) red_ss[row] = 1.0f / sqrtf(tot / (float)p.K + p.eps);
                }
            }
        }
        // this thread's epilogue items: (unit, token) pairs, token fastest among the M live tokens.  For a residual
        // update the old value and the next gain are fetched now, long before the epilogue needs them.
        static_assert(NCW * GBN * NX * 32 * RW * 4 <= RED_BYTES, "the batch-end sums fit the reduction buffer");
        const int gshift = s.swiglu ? 3 : 4, total = (ng << gshift) * p.M;
        constexpr int ITEMS = GBN * 16 * 8 * NB / (NCW * 32);
        float xold[ITEMS], gnext[ITEMS];
#pragma unroll
        for (int it4 = 0; it4 < ITEMS; ++it4) {
            xold[it4] = 0.f; gnext[it4] = 1.f;
            const int idx = tid + it4 * (NCW * 32);
            if (p.epi == EPI_ADD && alive && idx < total) {
                const int n = idx % p.M, ur = idx / p.M, gi = ur >> gshift, rr = ur & ((1 << gshift) - 1);
                if (rr < s.group_size(g0 + gi)) {
                    const int u = s.u_lo + s.group_lo(g0 + gi) + rr;
                    xold[it4] = __ldcg(p.y + (size_t)n * p.units + u);
                    if (p.next_gain) gnext[it4] = __ldg(p.next_gain + u);
                }
            }
        }
        for (int kt = 0; kt < s.n_kt; ++kt) {
            const bool slot_valid = kt * NCW + warp < nslots;
            uint32_t bf[NX][NTM][KSTEPS][2];                  // operand registers: block, term, k-step, (b0, b1)
#pragma unroll
            for (int nb = 0; nb < NX; ++nb)
#pragma unroll
                for (int t = 0; t < NTM; ++t)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        bf[nb][t][2 * q][0] = nx[nb][t][q].x; bf[nb][t][2 * q][1] = nx[nb][t][q].y;
                        bf[nb][t][2 * q + 1][0] = nx[nb][t][q].z; bf[nb][t][2 * q + 1][1] = nx[nb][t][q].w;
                    }
            if (kt + 1 < s.n_kt) fetch(kt + 1);
#pragma unroll
            for (int gi = 0; gi < GBN; ++gi) {
                if (gi >= ng) break;
                if (alive) alive = mbar_wait(&r.full_w[ws], it & 1, r.abort_flag, r.err, 5);
                if (alive && slot_valid) {
                    const uint32_t base = smem_u32(r.wring + ws * WSTAGE) + lm_row * WPITCH + (warp * SLOT + lm_col) * 2;
                    // independent accumulator chains: block x term x parity of the k-step; smallest terms are added first
                    float tc[NX][NTM][2][4] = {};
#pragma unroll
                    for (int j = 0; j < KSTEPS; ++j) {
                        uint32_t a0, a1, a2, a3;
                        ldmatrix_x4(base + j * 32, a0, a1, a2, a3);
#pragma unroll
                        for (int nb = 0; nb < NX; ++nb)
#pragma unroll
                            for (int t = NTM - 1; t >= 0; --t)
                                mma_bf16(tc[nb][t][j & 1], a0, a1, a2, a3, bf[nb][t][j][0], bf[nb][t][j][1]);
                    }
                    if (PAIRED) {
                        // registers 0 / 1 = hi / lo part of (unit g8, row 4 nb + t4), 2 / 3 = of (unit g8 + 8, same row): the sum of the
                        // lo products first, then the hi products, as in the unpaired form; acc[..][0], [1] = the two units
                        static_assert(NTERM == 2, "the paired form packs two terms");
#pragma unroll
                        for (int nb = 0; nb < NX; ++nb)
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                float sum = tc[nb][0][0][2 * h + 1] + tc[nb][0][1][2 * h + 1];
                                sum += tc[nb][0][0][2 * h] + tc[nb][0][1][2 * h];
                                acc[gi][nb][h] += sum;
                            }
                    } else {
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float sum = tc[nb][NTM - 1][0][e] + tc[nb][NTM - 1][1][e];
#pragma unroll
                                for (int t = NTM - 2; t >= 0; --t) sum += tc[nb][t][0][e] + tc[nb][t][1][e];
                                acc[gi][nb][e] += sum;
                            }
                    }
                }
                __syncwarp();
                if (alive && lane == 0) mbar_arrive(&r.empty_w[ws]);
                ++w_use;
                if (++ws == WS) { ws = 0; ++it; }
            }
        }
        // ---- batch end: partial sums of the 8 column slots meet in shared memory, in warp order ----
#pragma unroll
        for (int gi = 0; gi < GBN; ++gi)
#pragma unroll
            for (int nb = 0; nb < NX; ++nb) {
                float *dst = red + ((((warp * GBN + gi) * NX + nb) * 32) + lane) * RW;
                if (PAIRED) *reinterpret_cast<float2 *>(dst) = make_float2(acc[gi][nb][0], acc[gi][nb][1]);
                else *reinterpret_cast<float4 *>(dst) = make_float4(acc[gi][nb][0], acc[gi][nb][1], acc[gi][nb][2], acc[gi][nb][3]);
            }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
        if (alive) {
#pragma unroll
            for (int it4 = 0; it4 < ITEMS; ++it4) {
                const int idx = tid + it4 * (NCW * 32);
                if (idx >= total) break;
                const int n = idx % p.M, ur = idx / p.M, gi = ur >> gshift, rr = ur & ((1 << gshift) - 1);
                if (rr >= s.group_size(g0 + gi)) continue;
                // token n sits in block n / 8, column n % 8; rows 0..7 of the tile: regs 0,1; rows 8..15: regs 2,3
                // where the eight warps left this item's partial sums.  Unpaired: lane (unit % 8, token / 2), register
                // (unit / 8) * 2 + token % 2; paired: lane (unit % 8, token), register unit / 8
                const int nb = PAIRED ? n >> 2 : n >> 3, n8 = PAIRED ? (n & 3) : (n & 7);
                const int src_lane = (rr & 7) * 4 + (PAIRED ? n8 : (n8 >> 1)), reg = PAIRED ? 0 : (n8 & 1);
                const int e0 = PAIRED ? (s.swiglu ? 0 : (rr >> 3)) : (s.swiglu ? reg : (rr >> 3) * 2 + reg);
                const int e1 = PAIRED ? 1 : 2 + reg;            // SwiGLU: the up row of the unit (tile rows 8..15)
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    const float *q = red + ((((w * GBN + gi) * NX + nb) * 32) + src_lane) * RW;
                    s0 += q[e0];
                    if (s.swiglu) s1 += q[e1];
                }
                const float ri = normed ? red_ss[n] : 1.0f;
                const int u = s.u_lo + s.group_lo(g0 + gi) + rr;
                float *yp = p.y + (size_t)n * p.units + u;
                if (s.swiglu) {
                    const float gt = s0 * ri, up = s1 * ri;
                    const float a = gt / (1.0f + expf(-gt)) * up;
                    if (p.ys) store_split(p.ys, p.units >> 7, n, u, a); else __stcg(yp, a);
                } else if (p.epi == EPI_ADD) {
                    const float v = xold[it4] + s0 * ri;
                    __stcg(yp, v);
                    if (p.ys) store_split(p.ys, p.units >> 7, n, u, v * gnext[it4]);
                    // leave v^2 where this thread alone read its first partial: warp n % 8 adds them up below
                    red[((((0 * GBN + gi) * NX + nb) * 32) + src_lane) * RW + e0] = v * v;
                } else {
                    __stcg(yp, s0 * ri);
                }
            }
        }
        if (p.ss_out) {
            asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
            if (alive) {
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    const int row = nb * 8 + warp;              // this warp adds up the squares of pass row `row`
                    if (row >= p.M) continue;
                    const int n8 = warp;
                    float part = 0.f;
                    for (int i = lane; i < (ng << gshift); i += 32) {
                        const int gi = i >> gshift, rr = i & ((1 << gshift) - 1);
                        if (rr < s.group_size(g0 + gi))
                            part += PAIRED ? red[((((0 * GBN + gi) * NX + (row >> 2)) * 32) + (rr & 7) * 4 + (row & 3)) * RW + (rr >> 3)]
                                           : red[((((0 * GBN + gi) * NX + nb) * 32) + (rr & 7) * 4 + (n8 >> 1)) * RW + (rr >> 3) * 2 + (n8 & 1)];
                    }
                    part = warp_sum(part);
                    ss_acc[nb] += part;
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    }
    if (p.ss_out && alive && lane == 0) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
            if (nb * 8 + warp < p.M) __stcg(p.ss_out + (size_t)(nb * 8 + warp) * n_cta + cta, ss_acc[nb]);
    }
}

}  // namespace stream
}  // namespace knnssd
