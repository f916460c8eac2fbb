// Anchor construction of the pre-inference stage (Sec. 4.1): the sampled last hidden vectors of all domains are
// clustered with K-means (Lloyd's iteration, as many clusters as domains), and each cluster's k members nearest to
// its centroid become its anchors (Eq. (2): the k smallest distances minimise the sum over size-k subsets).
//
// The points are fp32 [N][d] (d = the model width, N = domains x samples per domain: 5 x 1000 in the paper's
// set-up, 100 MB at d = 5120); distances, sums and centroids are fp64, so that the integer decisions (nearest
// centroid, nearest members) do not hinge on fp32 rounding.  A round reads the points twice (assignment, centroid
// sums): both kernels are bound by that traffic.  Every reduction has a fixed order: results do not depend on timing.
#pragma once

#include "kernels.cuh"

namespace knnssd {
namespace anchors {

constexpr int MAXC = 16;       // most clusters (domains)
constexpr int CHUNK = 256;     // columns of the centroids staged in shared memory per step
constexpr int PTS = 8;         // points per block of assign_kernel: one per warp

// For each point: the squared distances to all n centroids; relabel != 0: labels[p] <- the nearest centroid (lowest
// index among equal distances), *changed set if that differs from the old label, counts[c] incremented; in both modes
// dist[p] <- the distance to the centroid of labels[p].  grid = ceil(N / PTS), 256 threads.
__global__ void __launch_bounds__(PTS * 32) assign_kernel(const float *__restrict__ x, int N, int d, const double *__restrict__ mu, int n,
                                                          int relabel, int *__restrict__ labels, double *__restrict__ dist,
                                                          int *__restrict__ counts, int *__restrict__ changed) {
    __shared__ double smu[MAXC][CHUNK];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p = blockIdx.x * PTS + warp;
    const bool live = p < N;
    double acc[MAXC];
#pragma unroll
    for (int c = 0; c < MAXC; ++c) acc[c] = 0.0;
    const float *xr = x + (size_t)(live ? p : 0) * d;
    for (int col0 = 0; col0 < d; col0 += CHUNK) {
        for (int idx = threadIdx.x; idx < n * CHUNK; idx += PTS * 32) {
            const int c = idx / CHUNK, j = idx % CHUNK;
            smu[c][j] = col0 + j < d ? mu[(size_t)c * d + col0 + j] : 0.0;
        }
        __syncthreads();
        if (live) {
            for (int j = lane; j < CHUNK && col0 + j < d; j += 32) {
                const double xv = (double)xr[col0 + j];
#pragma unroll
                for (int c = 0; c < MAXC; ++c)
                    if (c < n) {
                        const double diff = xv - smu[c][j];
                        acc[c] = fma(diff, diff, acc[c]);
                    }
            }
        }
        __syncthreads();
    }
    if (!live) return;
#pragma unroll
    for (int c = 0; c < MAXC; ++c)
        if (c < n) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        }
    if (lane == 0) {
        int best = labels[p];
        if (relabel) {
            best = 0;
            double bv = acc[0];
#pragma unroll
            for (int c = 1; c < MAXC; ++c)
                if (c < n && acc[c] < bv) { bv = acc[c]; best = c; }
            if (best != labels[p]) { labels[p] = best; atomicOr(changed, 1); }
            atomicAdd(counts + best, 1);
        }
        double own = acc[0];
#pragma unroll
        for (int c = 1; c < MAXC; ++c)
            if (c == best) own = acc[c];
        dist[p] = sqrt(own);
    }
}

// part[s][c][j] = sum of x[p][j] over the points p of slice s (S slices of `per` consecutive points) labelled c, added
// in index order.  grid = (ceil(d / 256), S), 256 threads: a thread owns one column.
__global__ void __launch_bounds__(256) partial_sums_kernel(const float *__restrict__ x, int N, int d, const int *__restrict__ labels,
                                                           int n, int per, double *__restrict__ part) {
    __shared__ double acc[MAXC][256];
    const int j = blockIdx.x * 256 + threadIdx.x, s = blockIdx.y;
    for (int c = 0; c < n; ++c) acc[c][threadIdx.x] = 0.0;
    const int p0 = s * per, p1 = min(N, p0 + per);
    if (j < d)
        for (int p = p0; p < p1; ++p) acc[labels[p]][threadIdx.x] += (double)x[(size_t)p * d + j];
    if (j < d)
        for (int c = 0; c < n; ++c) part[((size_t)s * n + c) * d + j] = acc[c][threadIdx.x];
}

// mu[c][j] = (sum over slices, in slice order, of part[s][c][j]) / counts[c]; a cluster without members keeps its
// centroid.  grid = (ceil(d / 256), n), 256 threads.
__global__ void fold_centroids_kernel(const double *__restrict__ part, const int *__restrict__ counts, int n, int d, int S,
                                      double *__restrict__ mu) {
    const int j = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y;
    if (j >= d || counts[c] == 0) return;
    double s = 0.0;
    for (int i = 0; i < S; ++i) s += part[((size_t)i * n + c) * d + j];
    mu[(size_t)c * d + j] = s / (double)counts[c];
}

// Eq. (2) for cluster c = blockIdx.x: k times, the not yet taken member with the smallest (distance, index);
// out[c][r] = its index, -1 once the cluster has run out of members.  taken[N] starts at zero.  256 threads.
__global__ void __launch_bounds__(256) select_anchors_kernel(const double *__restrict__ dist, const int *__restrict__ labels, int N, int k,
                                                             unsigned char *__restrict__ taken, int *__restrict__ out) {
    __shared__ double sv[256];
    __shared__ int si[256];
    const int c = blockIdx.x, tid = threadIdx.x;
    for (int r = 0; r < k; ++r) {
        double bv = INFINITY;
        int bi = -1;
        for (int p = tid; p < N; p += 256)
            if (labels[p] == c && !taken[p] && (bi < 0 || dist[p] < bv)) { bv = dist[p]; bi = p; }   // ascending p: first of equals wins
        sv[tid] = bv;
        si[tid] = bi;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (tid < o) {
                const double ov = sv[tid + o];
                const int oi = si[tid + o];
                if (oi >= 0 && (si[tid] < 0 || ov < sv[tid] || (ov == sv[tid] && oi < si[tid]))) { sv[tid] = ov; si[tid] = oi; }
            }
            __syncthreads();
        }
        if (tid == 0) {
            out[c * k + r] = si[0];
            if (si[0] >= 0) taken[si[0]] = 1;
        }
        __syncthreads();
    }
}

}  // namespace anchors
}  // namespace knnssd
