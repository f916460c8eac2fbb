// Host side of the tensor-core prompt pass: TMA tensor maps and the launches of prefill.cuh's kernels.
#pragma once

#include "prefill.cuh"

#include <cuda_runtime.h>

namespace knnssd {
namespace prefill {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link against the driver).
inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Map of a row-major bf16 matrix [rows][cols] (cols a multiple of 64) read in boxes of box_rows rows x 64 columns,
// 128-byte swizzle; rows past the end read as zero.
inline bool make_map(CUtensorMap *m, const void *base, size_t rows, size_t cols, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The contraction kernels need more dynamic shared memory than the default limit; the attribute belongs to the
// current device, so it is set once per device (one process may drive several GPUs).
inline bool gemm_attrs_once() {
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (done[dev]) return true;
    const bool ok =
        cudaFuncSetAttribute(gemm_split_kernel<PF_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(gemm_split_kernel<PF_ADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(gemm_split_kernel<PF_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(gemm_split_kernel<PF_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(gemm_wide_kernel<PF_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, WIDE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(gemm_wide_kernel<PF_ADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, WIDE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(attn_prompt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem_bytes<128>()) == cudaSuccess &&
        cudaFuncSetAttribute(attn_prompt_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem_bytes<64>()) == cudaSuccess;
    done[dev] = ok;
    return ok;
}

// Accumulator columns per tile.  gemm_split_kernel runs one CTA per SM that walks the tiles round after round;
// gemm_wide_kernel one CTA per tile.  The main loop is bound by shared-memory traffic (measured per k-block and CTA:
// 0.57 / 0.69 / 0.81 us at 128 / 192 / 256 columns, 1.1 - 1.4 at 2 x 160): per k-block TMA writes the two activation
// planes (32 KB) and bn / 8 KB of weights, and the tensor core reads the planes once and the weights twice (hi and lo
// products), 64 + 3 bn / 8 KB in all; the 320-column tiles of gemm_wide_kernel (returned as WIDE_BN; store and add
// epilogues only) read the planes once per half and are charged 15 % on top, as measured, plus ~10 us per round for the
// prologue and epilogue that nothing overlaps there (1960 KB at that rate; the walking kernel pays ~3 us once).  The
// width with the lowest rounds x traffic x k-blocks + fixed cost wins (ties: the wider tile).
inline int pick_bn(int T, int N, int K, bool swiglu, int n_sms) {
    const int row_tiles = (T + BM - 1) / BM;
    const long nkb = K / BK;
    int best = 0;
    long best_cost = 0;
    for (int bn = BOX_N; bn <= (swiglu ? BN_MAX : WIDE_BN); bn += BOX_N) {
        if (bn > BN_MAX && bn != WIDE_BN) continue;
        if (swiglu && bn % 128) continue;
        const int per = swiglu ? bn / 2 : bn;
        const long ctas = (long)row_tiles * ((N + per - 1) / per);
        const long traffic = bn == WIDE_BN ? 248 : 64 + 3 * bn / 8;
        const long rounds = (ctas + n_sms - 1) / n_sms;
        const long cost = bn == WIDE_BN ? rounds * (traffic * nkb + 1960) : rounds * traffic * nkb + 600;
        if (!best || cost <= best_cost) { best = bn; best_cost = cost; }
    }
    return best;
}

// One contraction over T rows.  `planes` = the activation map (hi rows [0, cap), lo rows [cap, 2 cap)); W0 (and W1 for
// SwiGLU: W0 = gate, W1 = up) are [N][K] bf16.  STORE with W1 and W2 given: the three matrices (nA, nB and nC rows, all
// multiples of BOX_N) are stacked along the output units, N = nA + nB + nC, one launch for q, k and v.
// Returns false if a tensor map could not be made.
// What the q / k / v launch needs to finish the heads in its epilogue (rotary embedding, K / V rows into the cache).
struct QkvFuse {
    const float2 *rope;    // [T][64]
    bf16_t *kc, *vc;
    int max_seq, pos0, head_dim;
};

// `fuse` (stacked q, k, v only): if the head dimension is 128 and the launch takes 256-column tiles, the epilogue does
// the rotary embedding and writes K / V to the cache itself; *fused says whether it did (otherwise the caller runs
// rope_kv_rows_kernel on y).
inline bool launch_gemm(const CUtensorMap &planes, int cap, const void *W0, const void *W1, int N, int K, int T, int epi, float *y,
                        int ldy, int col0, bf16_t *out_hi, bf16_t *out_lo, int ldo, int *err, int n_sms, cudaStream_t s,
                        const void *W2 = nullptr, int nA = 0, int nB = 0, const QkvFuse *fuse = nullptr, bool *fused = nullptr,
                        const float *row_scale = nullptr) {
    if (fused) *fused = false;
    if (!gemm_attrs_once()) return false;
    CUtensorMap tb0, tb1, tb2;
    const bool stacked = epi == PF_STORE && W1 && W2;
    if (!make_map(&tb0, W0, (size_t)(stacked ? nA : N), (size_t)K, BOX_N)) return false;
    if (epi == PF_SWIGLU) {
        if (!make_map(&tb1, W1, (size_t)N, (size_t)K, BOX_N)) return false;
        tb2 = tb1;
    } else if (stacked) {
        if (!make_map(&tb1, W1, (size_t)nB, (size_t)K, BOX_N) || !make_map(&tb2, W2, (size_t)(N - nA - nB), (size_t)K, BOX_N)) return false;
    } else {
        tb1 = tb0;
        tb2 = tb0;
    }
    const int bn = pick_bn(T, N, K, epi == PF_SWIGLU, n_sms);
    const int per = epi == PF_SWIGLU ? bn / 2 : bn;
    const dim3 grid((T + BM - 1) / BM, (N + per - 1) / per);
    GemmArgs g{T, K, N, bn, y, ldy, col0, out_hi, out_lo, ldo, err, (int)grid.x, (int)grid.y, stacked ? nA : N, stacked ? nB : 0,
               row_scale, nullptr, nullptr, nullptr, 0, 0};
    // gemm_split_kernel: one CTA per SM walks the tiles (the epilogue of a tile runs under the next tile's products)
    const int n_tiles = (int)(grid.x * grid.y);
    const dim3 pgrid(n_tiles < n_sms ? n_tiles : n_sms);
    const bool fuse_heads = stacked && fuse && fuse->head_dim == 128 && bn == 256 && nA % 128 == 0 && nB % 128 == 0 && N % 128 == 0;
    if (fuse_heads) { g.rope = fuse->rope; g.kc = fuse->kc; g.vc = fuse->vc; g.max_seq = fuse->max_seq; g.pos0 = fuse->pos0; }
    if (fuse_heads) {
        gemm_split_kernel<PF_QKV><<<pgrid, GEMM_THREADS, GEMM_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
        if (fused) *fused = true;
    } else if (bn == WIDE_BN && epi == PF_STORE) gemm_wide_kernel<PF_STORE><<<grid, GEMM_THREADS, WIDE_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
    else if (bn == WIDE_BN) gemm_wide_kernel<PF_ADD><<<grid, GEMM_THREADS, WIDE_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
    else if (epi == PF_STORE) gemm_split_kernel<PF_STORE><<<pgrid, GEMM_THREADS, GEMM_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
    else if (epi == PF_ADD) gemm_split_kernel<PF_ADD><<<pgrid, GEMM_THREADS, GEMM_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
    else gemm_split_kernel<PF_SWIGLU><<<pgrid, GEMM_THREADS, GEMM_SMEM, s>>>(planes, tb0, tb1, tb2, g, cap);
    return true;
}

}  // namespace prefill
}  // namespace knnssd
