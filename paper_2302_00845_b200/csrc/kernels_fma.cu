// FMA-pipe kernels for m <= 16 workers (any dtype, d a multiple of 4).
//
// Every thread owns groups of 4 consecutive columns and keeps the whole upper triangle of
// G = C^T C plus b = C^T r in registers (M(M+1)/2 + M accumulators), so each loaded
// gradient element is used from registers and nothing is staged in shared memory.
//
//   gram_fma_kernel    multi-block pass 1 of the two-pass formulation
//   fma_combine_kernel fixed-order fp64 sum of the block partials -> G, b
//   fused_step_kernel  one CTA does the whole step (Gram, the m decisions of Algorithm 6,
//                      permutation slots of Algorithm 7, update of r): the step's inputs
//                      come from HBM once and are re-read from cache for the update
//   fused_step_cluster_kernel  the same step on a thread-block cluster (DSMEM reduction)
//   fused_logreg_step_kernel   the step straight from logistic-regression feature rows
//   gram_fma_tma_kernel        TMA-fed pass 1 for long rows; its last CTA combines and decides
#include <cooperative_groups.h>
#include <stdlib.h>

#include "common.cuh"
#include "scan.cuh"

namespace cg = cooperative_groups;

template <int M>
struct Tri {
  static constexpr int NPAIR = M * (M + 1) / 2;
  static constexpr int NACC = NPAIR + M;
  static constexpr int Q = (NACC + 31) / 32;  // values per lane after the warp reduction
  static constexpr int NPAD = 32 * Q;
  __host__ __device__ static constexpr int idx(int a, int b) {  // a <= b
    return a * M - a * (a - 1) / 2 + (b - a);
  }
};

template <typename T>
__device__ __forceinline__ void ld4(const T *p, float (&v)[4]);
template <>
__device__ __forceinline__ void ld4<float>(const float *p, float (&v)[4]) {
  const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <>
__device__ __forceinline__ void ld4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[4]) {
  const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
  v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
  v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
}
// r is written later in the fused kernel, so it is read with ordinary (coherent) loads
__device__ __forceinline__ void ld4_r(const float *p, float (&v)[4]) {
  const float4 q = *reinterpret_cast<const float4 *>(p);
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}

// accumulate the Gram contributions of column groups v0, v0+vstride, ... < nvec
template <typename T, int M>
__device__ __forceinline__ void gram_accumulate(const T *__restrict__ g, const float *r, int m,
                                                long long d, long long v0, long long vstride,
                                                long long nvec, float (&acc)[Tri<M>::NPAD]) {
  const size_t slab = (size_t)m * (size_t)d;
  for (long long v = v0; v < nvec; v += vstride) {
    const size_t x = (size_t)v * 4;
    float c[M][4];
#pragma unroll
    for (int i = 0; i < M; ++i) {
      if (i < m) {
        float a[4], b[4];
        ld4<T>(g + (size_t)i * (size_t)d + x, a);
        ld4<T>(g + slab + (size_t)i * (size_t)d + x, b);
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = a[j] - b[j];  // c = z1 - z2
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = 0.f;
      }
    }
    float rv[4];
    ld4_r(r + x, rv);
#pragma unroll
    for (int a = 0; a < M; ++a) {
#pragma unroll
      for (int b = a; b < M; ++b) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          acc[Tri<M>::idx(a, b)] = fmaf(c[a][j], c[b][j], acc[Tri<M>::idx(a, b)]);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        acc[Tri<M>::NPAIR + a] = fmaf(rv[j], c[a][j], acc[Tri<M>::NPAIR + a]);
    }
  }
}

// Sum a vector of N = 32*Q values across the warp with N - Q shuffles: in the round with
// lane distance `half` the lanes whose bit `half` is set keep the upper half of the entries
// still alive, the others the lower half, and each adds what its partner sends.  Afterwards
// lane L holds in v[0..Q) the totals of entries q + Q*L.  The addition tree is fixed.
template <int N>
__device__ __forceinline__ void warp_reduce_vec(float (&v)[N], int lane) {
  int cnt = N / 2;
#pragma unroll
  for (int half = 16; half >= 1; half >>= 1) {
    const bool upper = (lane & half) != 0;
#pragma unroll
    for (int j = 0; j < N / 2; ++j) {
      if (j < cnt) {
        const float send = upper ? v[j] : v[j + cnt];
        const float keep = upper ? v[j + cnt] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, half);
      }
    }
    cnt >>= 1;
  }
}

// block-level: every warp reduces, warp totals go to smem as double, thread e < NACC adds the
// warps in index order.  Returns the block total of entry threadIdx.x (valid for tid < NACC).
template <int M, int WARPS>
__device__ __forceinline__ double block_reduce_acc(float (&acc)[Tri<M>::NPAD], double *red /*[WARPS][NPAD]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  warp_reduce_vec<Tri<M>::NPAD>(acc, lane);
#pragma unroll
  for (int q = 0; q < Tri<M>::Q; ++q) red[warp * Tri<M>::NPAD + q + Tri<M>::Q * lane] = (double)acc[q];
  __syncthreads();
  double v = 0.0;
  if (threadIdx.x < Tri<M>::NACC) {
    for (int w = 0; w < WARPS; ++w) v += red[w * Tri<M>::NPAD + threadIdx.x];
  }
  return v;
}

// ------------------------------------------------------------------------------------
template <typename T, int M>
__global__ void __launch_bounds__(256)
gram_fma_kernel(const T *__restrict__ g, const float *__restrict__ r, int m, long long d,
                double *__restrict__ partials) {
  float acc[Tri<M>::NPAD];
#pragma unroll
  for (int e = 0; e < Tri<M>::NPAD; ++e) acc[e] = 0.f;
  gram_accumulate<T, M>(g, r, m, d, (long long)blockIdx.x * blockDim.x + threadIdx.x,
                        (long long)gridDim.x * blockDim.x, d / 4, acc);
  __shared__ double red[8 * Tri<M>::NPAD];
  const double v = block_reduce_acc<M, 8>(acc, red);
  if (threadIdx.x < Tri<M>::NACC) partials[(size_t)blockIdx.x * Tri<M>::NACC + threadIdx.x] = v;
}

// 6 slices of the block list are summed side by side (slice p takes blocks p, p+6, ...), then
// the slices are added in index order: fixed order for a fixed grid.
template <int M>
__global__ void __launch_bounds__(6 * Tri<M>::NPAD)
fma_combine_kernel(const double *__restrict__ partials, int blocks, int m, double *__restrict__ gram) {
  __shared__ double part[6][Tri<M>::NPAD];
  const int e = threadIdx.x % Tri<M>::NPAD, slice = threadIdx.x / Tri<M>::NPAD;
  double v = 0.0;
  if (e < Tri<M>::NACC)
    for (int b = slice; b < blocks; b += 6) v += partials[(size_t)b * Tri<M>::NACC + e];
  part[slice][e] = v;
  __syncthreads();
  if (slice != 0 || e >= Tri<M>::NACC) return;
  v = 0.0;
#pragma unroll
  for (int p = 0; p < 6; ++p) v += part[p][e];
  if (e < Tri<M>::NPAIR) {
    int a = 0, rem = e;
    while (rem >= M - a) { rem -= M - a; ++a; }
    const int bcol = a + rem;
    if (a < m && bcol < m) {
      gram[(size_t)a * m + bcol] = v;
      gram[(size_t)bcol * m + a] = v;
    }
  } else {
    const int a = e - Tri<M>::NPAIR;
    if (a < m) gram[(size_t)m * m + a] = v;
  }
}

// Decisions of the single-launch kernels: Algorithm 6 for i = 0..m-1 on
// t_i = b_i + sum_{k<i} s_k G_ki from the block totals (triangle entries, then b), signs /
// margins / permutation slots (Algorithm 7) written out.  The block totals are spread into the
// scan's shared arrays (full G, b, the current pairs fetched by 2m threads at once), warp 0
// takes the decisions with the chain in registers, the block writes out, and the signs land
// in ssh as +-1.0f.  (A one-thread loop paid two dependent global loads per worker.)
template <int M>
__device__ __forceinline__ void fused_decide_block(const double *tot, double *scan_sh, int m, int n, int k,
                                                   const int32_t *__restrict__ perm_cur,
                                                   int32_t *__restrict__ perm_next, int8_t *__restrict__ signs,
                                                   float *__restrict__ margins, double *__restrict__ rnorm2,
                                                   int *__restrict__ status, const CdgRule &rule, float *ssh,
                                                   bool write_out) {
  const ScanSmem S = scan_smem(scan_sh, m);
  if (threadIdx.x < Tri<M>::NACC) {
    const int e = threadIdx.x;
    const double v = tot[e];
    if (e < Tri<M>::NPAIR) {
      int a = 0, rem = e;
      while (rem >= M - a) { rem -= M - a; ++a; }
      const int b = a + rem;
      if (a < m && b < m) { S.g[a * m + b] = v; S.g[b * m + a] = v; }
    } else {
      const int a = e - Tri<M>::NPAIR;
      if (a < m) S.t[a] = v;
    }
  }
  scan_load_pairs(S, perm_cur, m, n, k);
  __syncthreads();
  scan_decide_and_write(S, S.g, m, n, k, perm_next, signs, margins, rnorm2, status, rule, -1.0, write_out);
  if (threadIdx.x < m) ssh[threadIdx.x] = (float)S.s[threadIdx.x];
  __syncthreads();
}

// ------------------------------------------------------------------------------------
// Whole step in one CTA.  The thread count shrinks with M so the accumulators stay in
// registers: 1024 threads for M = 4, 512 for M = 8, 256 for M = 16.
// ------------------------------------------------------------------------------------
template <int M>
struct FusedCfg { static constexpr int THREADS = (M <= 4) ? 1024 : (M <= 8 ? 512 : 256); };

template <typename T, int M>
__global__ void __launch_bounds__(FusedCfg<M>::THREADS)
fused_step_kernel(const T *__restrict__ g, float *r, int m, int n, long long d, int k, int count,
                  const int32_t *__restrict__ perm_cur, int32_t *__restrict__ perm_next,
                  int8_t *__restrict__ signs, float *__restrict__ margins,
                  double *__restrict__ rnorm2, int *__restrict__ status, const CdgRule rule) {
  extern __shared__ double dsh[];
  constexpr int WARPS = FusedCfg<M>::THREADS / 32;
  double *red = dsh;                                  // [WARPS][NPAD]
  double *tot = red + WARPS * Tri<M>::NPAD;           // [NPAD]
  double *scan_sh = tot + Tri<M>::NPAD;               // [4M + M*M] the scan's arrays
  float *ssh = reinterpret_cast<float *>(scan_sh + 4 * M + M * M);  // [M]
  cdg_grid_dep_wait();            // r comes from the step before, the rows from the caller's last launch

  // `count` consecutive steps ([count][2][m][d] rows): r stays in this SM's cache between them
  const long long nvec = d / 4;
  for (int kk = 0; kk < count; ++kk, ++k, g += 2 * (size_t)m * (size_t)d) {
  float acc[Tri<M>::NPAD];
#pragma unroll
  for (int e = 0; e < Tri<M>::NPAD; ++e) acc[e] = 0.f;
  gram_accumulate<T, M>(g, r, m, d, threadIdx.x, blockDim.x, nvec, acc);
  const double v = block_reduce_acc<M, WARPS>(acc, red);
  if (threadIdx.x < Tri<M>::NACC) tot[threadIdx.x] = v;
  __syncthreads();
  fused_decide_block<M>(tot, scan_sh, m, n, k, perm_cur, perm_next, signs, margins, rnorm2, status, rule, ssh, true);

  // r <- r + sum_i s_i c_i (i ascending), inputs re-read through the cache
  const size_t slab = (size_t)m * (size_t)d;
  for (long long vv = threadIdx.x; vv < nvec; vv += blockDim.x) {
    const size_t x = (size_t)vv * 4;
    float rv[4];
    ld4_r(r + x, rv);
    double a4[4] = {(double)rv[0], (double)rv[1], (double)rv[2], (double)rv[3]};
#pragma unroll
    for (int i = 0; i < M; ++i) {
      if (i < m) {
        float a[4], b[4];
        ld4<T>(g + (size_t)i * (size_t)d + x, a);
        ld4<T>(g + slab + (size_t)i * (size_t)d + x, b);
        const float s = ssh[i];
#pragma unroll
        for (int j = 0; j < 4; ++j) a4[j] += (double)(s * (a[j] - b[j]));
      }
    }
    *reinterpret_cast<float4 *>(r + x) =
        make_float4((float)a4[0], (float)a4[1], (float)a4[2], (float)a4[3]);
  }
  __syncthreads();   // the new r and the shared arrays are settled before the next step reads them
  }
}

// ------------------------------------------------------------------------------------
// The same step spread over a thread-block cluster: CTA `rank` of C takes every C-th group of
// columns, the C block totals of the Gram entries meet through distributed shared memory (each
// CTA adds them in rank order, so all hold the same sums), every CTA takes the same decisions,
// rank 0 writes them out, and each CTA updates the columns it read.  C SMs' worth of loads in
// flight and of cache bandwidth instead of one; two cluster barriers per step.
// ------------------------------------------------------------------------------------
template <int M>
struct ClusterCfg { static constexpr int THREADS = (M <= 8) ? 128 : 256; };   // >= the Gram entries of M

template <typename T, int M>
__global__ void __launch_bounds__(ClusterCfg<M>::THREADS)
fused_step_cluster_kernel(const T *__restrict__ g, float *r, int m, int n, long long d, int k, int count,
                          const int32_t *__restrict__ perm_cur, int32_t *__restrict__ perm_next,
                          int8_t *__restrict__ signs, float *__restrict__ margins,
                          double *__restrict__ rnorm2, int *__restrict__ status, const CdgRule rule) {
  extern __shared__ double dsh[];
  constexpr int WARPS = ClusterCfg<M>::THREADS / 32;
  double *red = dsh;                                  // [WARPS][NPAD]
  double *mine = red + WARPS * Tri<M>::NPAD;          // [NPAD] this CTA's totals, read by the whole cluster
  double *tot = mine + Tri<M>::NPAD;                  // [NPAD] totals of the cluster
  double *scan_sh = tot + Tri<M>::NPAD;               // [4M + M*M] the scan's arrays
  float *ssh = reinterpret_cast<float *>(scan_sh + 4 * M + M * M);  // [M]
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster.block_rank(), csize = cluster.num_blocks();
  cdg_grid_dep_wait();            // r comes from the step before, the rows from the caller's last launch

  const long long nvec = d / 4;
  const long long v0 = (long long)rank * blockDim.x + threadIdx.x, vstride = (long long)csize * blockDim.x;
  const size_t slab = (size_t)m * (size_t)d;
  for (int kk = 0; kk < count; ++kk, ++k, g += 2 * slab) {
    float acc[Tri<M>::NPAD];
#pragma unroll
    for (int e = 0; e < Tri<M>::NPAD; ++e) acc[e] = 0.f;
    gram_accumulate<T, M>(g, r, m, d, v0, vstride, nvec, acc);
    const double v = block_reduce_acc<M, WARPS>(acc, red);
    if (threadIdx.x < Tri<M>::NACC) mine[threadIdx.x] = v;
    cluster.sync();                                   // every CTA's totals are in place
    if (threadIdx.x < Tri<M>::NACC) {
      double sum = 0.0;
      for (unsigned c = 0; c < csize; ++c) sum += cluster.map_shared_rank(mine, c)[threadIdx.x];
      tot[threadIdx.x] = sum;
    }
    cluster.sync();                                   // all remote reads done: `mine` may be rewritten
    fused_decide_block<M>(tot, scan_sh, m, n, k, perm_cur, perm_next, signs, margins, rnorm2, status, rule, ssh,
                          rank == 0);

    // r <- r + sum_i s_i c_i (i ascending) on this CTA's columns, inputs re-read through the cache
    for (long long vv = v0; vv < nvec; vv += vstride) {
      const size_t x = (size_t)vv * 4;
      float rv[4];
      ld4_r(r + x, rv);
      double a4[4] = {(double)rv[0], (double)rv[1], (double)rv[2], (double)rv[3]};
#pragma unroll
      for (int i = 0; i < M; ++i) {
        if (i < m) {
          float a[4], b[4];
          ld4<T>(g + (size_t)i * (size_t)d + x, a);
          ld4<T>(g + slab + (size_t)i * (size_t)d + x, b);
          const float s = ssh[i];
#pragma unroll
          for (int j = 0; j < 4; ++j) a4[j] += (double)(s * (a[j] - b[j]));
        }
      }
      *reinterpret_cast<float4 *>(r + x) =
          make_float4((float)a4[0], (float)a4[1], (float)a4[2], (float)a4[3]);
    }
    __syncthreads();   // the shared arrays are settled before the next step reuses them
  }
}

// ------------------------------------------------------------------------------------
// Logistic regression without a gradient buffer: the whole step from the feature rows.
// For worker i the pair's items are p = perm_cur[i][2k], q = perm_cur[i][2k+1]; with
// a = sigma(<w,x_p>) - y_p and b = sigma(<w,x_q>) - y_q the difference is c_i = a x_p - b x_q
// (each product rounded to fp32 like a stored gradient would be).  One CTA: coefficients,
// Gram, decisions, update.
// ------------------------------------------------------------------------------------
template <int M>
__device__ __forceinline__ void logreg_diffs(const float *__restrict__ X, const size_t *rowoff, const float *coef,
                                             int m, size_t x, float (&c)[M][4]) {
#pragma unroll
  for (int i = 0; i < M; ++i) {
    if (i < m) {
      float xp[4], xq[4];
      ld4<float>(X + rowoff[i] + x, xp);
      ld4<float>(X + rowoff[m + i] + x, xq);
#pragma unroll
      for (int j = 0; j < 4; ++j) c[i][j] = __fsub_rn(__fmul_rn(coef[i], xp[j]), __fmul_rn(coef[m + i], xq[j]));
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) c[i][j] = 0.f;
    }
  }
}

// Runs as a cluster of C >= 1 CTAs: CTA `rank` takes every C-th group of columns; the 2m dot
// products and the Gram entries are summed over the cluster through distributed shared memory in
// rank order, so every CTA holds the same coefficients and takes the same decisions.
template <int M, int THREADS>
__global__ void __launch_bounds__(THREADS)
fused_logreg_step_kernel(const float *__restrict__ X, const float *__restrict__ y, const float *__restrict__ w,
                         float *r, int m, int n, long long d, int k, const int32_t *__restrict__ perm_cur,
                         int32_t *__restrict__ perm_next, int8_t *__restrict__ signs, float *__restrict__ margins,
                         double *__restrict__ rnorm2, int *__restrict__ status, const CdgRule rule) {
  extern __shared__ double dsh[];
  constexpr int WARPS = THREADS / 32;
  double *red = dsh;                                  // [WARPS][NPAD]; first used as [WARPS][2M] for the dots
  double *mine = red + WARPS * Tri<M>::NPAD;          // [NPAD] this CTA's totals, read by the whole cluster
  double *tot = mine + Tri<M>::NPAD;                  // [NPAD] totals of the cluster
  double *dots = tot + Tri<M>::NPAD;                  // [2M] this CTA's share of <w, x>, read by the cluster
  double *scan_sh = dots + 2 * M;                     // [4M + M*M] the scan's arrays
  float *ssh = reinterpret_cast<float *>(scan_sh + 4 * M + M * M);  // [M]
  float *coef = ssh + M;                              // [2M]: a_0..a_{m-1}, b_0..b_{m-1}
  float *yv = coef + 2 * M;                           // [2M]
  size_t *rowoff = reinterpret_cast<size_t *>(yv + 2 * M);      // [2M] element offsets of the rows in X
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster.block_rank(), csize = cluster.num_blocks();
  const long long nvec = d / 4;
  const long long v0 = (long long)rank * THREADS + threadIdx.x, vstride = (long long)csize * THREADS;
  cdg_grid_dep_wait();            // r and the current order come from earlier launches

  if (threadIdx.x < 2 * m) {
    const int q = threadIdx.x / m, i = threadIdx.x % m;
    const int item = perm_cur[(size_t)i * n + 2 * k + q];
    rowoff[threadIdx.x] = ((size_t)i * n + item) * (size_t)d;
    yv[threadIdx.x] = y[(size_t)i * n + item];
  }
  __syncthreads();

  // <w, x> for the 2m rows
  {
    float z[2 * M];
#pragma unroll
    for (int e = 0; e < 2 * M; ++e) z[e] = 0.f;
    for (long long v = v0; v < nvec; v += vstride) {
      const size_t x = (size_t)v * 4;
      float wv[4];
      ld4<float>(w + x, wv);
#pragma unroll
      for (int e = 0; e < 2 * M; ++e) {
        if (e < 2 * m) {
          float xv[4];
          ld4<float>(X + rowoff[e] + x, xv);
#pragma unroll
          for (int j = 0; j < 4; ++j) z[e] = fmaf(wv[j], xv[j], z[e]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 2 * M; ++e) {
      double v = (double)z[e];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
      if (lane == 0) red[warp * 2 * M + e] = v;
    }
  }
  __syncthreads();
  if (threadIdx.x < 2 * m) {
    double zz = 0.0;
    for (int wi = 0; wi < WARPS; ++wi) zz += red[wi * 2 * M + threadIdx.x];
    dots[threadIdx.x] = zz;
  }
  cluster.sync();
  if (threadIdx.x < 2 * m) {
    double zz = 0.0;
    for (unsigned c = 0; c < csize; ++c) zz += cluster.map_shared_rank(dots, c)[threadIdx.x];
    const float zf = (float)zz;
    // sigma(z) - y without cancellation for y in {0,1}: sigma(z) - 1 = -sigma(-z)
    coef[threadIdx.x] = (yv[threadIdx.x] > 0.5f) ? -1.f / (1.f + expf(zf)) : 1.f / (1.f + expf(-zf));
  }
  __syncthreads();

  float acc[Tri<M>::NPAD];
#pragma unroll
  for (int e = 0; e < Tri<M>::NPAD; ++e) acc[e] = 0.f;
  for (long long v = v0; v < nvec; v += vstride) {
    const size_t x = (size_t)v * 4;
    float c[M][4], rv[4];
    logreg_diffs<M>(X, rowoff, coef, m, x, c);
    ld4_r(r + x, rv);
#pragma unroll
    for (int a = 0; a < M; ++a) {
#pragma unroll
      for (int b = a; b < M; ++b) {
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[Tri<M>::idx(a, b)] = fmaf(c[a][j], c[b][j], acc[Tri<M>::idx(a, b)]);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[Tri<M>::NPAIR + a] = fmaf(rv[j], c[a][j], acc[Tri<M>::NPAIR + a]);
    }
  }
  const double v = block_reduce_acc<M, WARPS>(acc, red);
  if (threadIdx.x < Tri<M>::NACC) mine[threadIdx.x] = v;
  cluster.sync();                                     // every CTA's totals are in place
  if (threadIdx.x < Tri<M>::NACC) {
    double sum = 0.0;
    for (unsigned c = 0; c < csize; ++c) sum += cluster.map_shared_rank(mine, c)[threadIdx.x];
    tot[threadIdx.x] = sum;
  }
  cluster.sync();                                     // remote reads done before any CTA moves on or leaves
  fused_decide_block<M>(tot, scan_sh, m, n, k, perm_cur, perm_next, signs, margins, rnorm2, status, rule, ssh,
                        rank == 0);

  for (long long vv = v0; vv < nvec; vv += vstride) {
    const size_t x = (size_t)vv * 4;
    float c[M][4], rv[4];
    logreg_diffs<M>(X, rowoff, coef, m, x, c);
    ld4_r(r + x, rv);
    double a4[4] = {(double)rv[0], (double)rv[1], (double)rv[2], (double)rv[3]};
#pragma unroll
    for (int i = 0; i < M; ++i) {
      if (i < m) {
        const float s = ssh[i];
#pragma unroll
        for (int j = 0; j < 4; ++j) a4[j] += (double)(s * c[i][j]);
      }
    }
    *reinterpret_cast<float4 *>(r + x) = make_float4((float)a4[0], (float)a4[1], (float)a4[2], (float)a4[3]);
  }
}

template <int M> struct ClusterCfg;
template <int M> static int fused_cluster_size(const cdgrab_ctx *h);

template <int M, int THREADS>
static cudaError_t launch_fused_logreg_tt(cdgrab_ctx *h, const float *X, const float *y, const float *w, int csize,
                                          cudaStream_t st) {
  constexpr int WARPS = THREADS / 32;
  const size_t smem = (WARPS * Tri<M>::NPAD + 2 * Tri<M>::NPAD + 2 * M + 4 * M + M * M) * sizeof(double) +
                      (M + 4 * M) * sizeof(float) + 2 * M * sizeof(size_t) + 16;
  static CdgPerDevice attr_set;
  if (const cudaError_t e = cdg_raise_smem_limit(attr_set, h->device, fused_logreg_step_kernel<M, THREADS>, smem);
      e != cudaSuccess)
    return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = csize; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = h->pdl ? 2 : 1;
  CdgProfScope ps(h, CDGRAB_K_FUSED, st);
  return cudaLaunchKernelEx(&cfg, fused_logreg_step_kernel<M, THREADS>, X, y, w, h->r, h->m, h->n, h->d, h->k,
                            (const int32_t *)h->perm_cur, h->perm_next, h->signs, h->margins, h->rnorm2, h->status,
                            cdg_rule_of(h));
}

template <int M>
static cudaError_t launch_fused_logreg_t(cdgrab_ctx *h, const float *X, const float *y, const float *w,
                                         cudaStream_t st);

cudaError_t cdg_launch_fused_logreg(cdgrab_ctx *h, const float *X, const float *y, const float *w, cudaStream_t st) {
  const int M = h->m <= 4 ? 4 : (h->m <= 8 ? 8 : 16);
  if (M == 4) return launch_fused_logreg_t<4>(h, X, y, w, st);
  if (M == 8) return launch_fused_logreg_t<8>(h, X, y, w, st);
  return launch_fused_logreg_t<16>(h, X, y, w, st);
}

// ------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------
static int pick_M(int m) { return m <= 4 ? 4 : (m <= 8 ? 8 : 16); }

bool cdg_fused_supported(int m, long long d, int dtype) {
  (void)dtype;
  return m <= 16 && d % 4 == 0;
}

// CTAs per cluster for the spread-out step: one per THREADS column groups, 4 or 8, else a single CTA
template <int M>
static int fused_cluster_size(const cdgrab_ctx *h) {
  if (h->cluster_off) return 1;
  const long long groups = (h->d / 4 + ClusterCfg<M>::THREADS - 1) / ClusterCfg<M>::THREADS;
  int c = 1;
  while (c < 8 && 2 * c <= groups) c *= 2;
  return c >= 4 ? c : 1;      // two CTAs do not pay for the cluster barriers (measured at d = 1024)
}

template <int M>
static cudaError_t launch_fused_logreg_t(cdgrab_ctx *h, const float *X, const float *y, const float *w,
                                         cudaStream_t st) {
  const int csize = fused_cluster_size<M>(h);
  if (csize > 1) return launch_fused_logreg_tt<M, ClusterCfg<M>::THREADS>(h, X, y, w, csize, st);
  return launch_fused_logreg_tt<M, FusedCfg<M>::THREADS>(h, X, y, w, 1, st);
}

template <typename T, int M>
static cudaError_t launch_fused_cluster_t(cdgrab_ctx *h, const void *grads, int count, int csize, cudaStream_t st) {
  constexpr int THREADS = ClusterCfg<M>::THREADS;
  const size_t smem = ((THREADS / 32) * Tri<M>::NPAD + 2 * Tri<M>::NPAD + 4 * M + M * M) * sizeof(double) +
                      M * sizeof(float);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = csize; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = h->pdl ? 2 : 1;
  CdgProfScope ps(h, CDGRAB_K_FUSED, st);
  return cudaLaunchKernelEx(&cfg, fused_step_cluster_kernel<T, M>, (const T *)grads, h->r, h->m, h->n, h->d, h->k,
                            count, (const int32_t *)h->perm_cur, h->perm_next, h->signs, h->margins, h->rnorm2,
                            h->status, cdg_rule_of(h));
}

template <typename T, int M>
static cudaError_t launch_fused_t(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st) {
  const int csize = fused_cluster_size<M>(h);
  if (csize > 1) return launch_fused_cluster_t<T, M>(h, grads, count, csize, st);
  const size_t smem = ((FusedCfg<M>::THREADS / 32) * Tri<M>::NPAD + Tri<M>::NPAD + 4 * M + M * M) * sizeof(double) +
                      M * sizeof(float);
  static CdgPerDevice attr_set;
  if (const cudaError_t e = cdg_raise_smem_limit(attr_set, h->device, fused_step_kernel<T, M>, smem); e != cudaSuccess)
    return e;
  {
    CdgProfScope ps(h, CDGRAB_K_FUSED, st);
    cdg_launch_dep(h, fused_step_kernel<T, M>, dim3(1), dim3(FusedCfg<M>::THREADS), smem, st, (const T *)grads, h->r,
                   h->m, h->n, h->d, h->k, count, h->perm_cur, h->perm_next, h->signs, h->margins, h->rnorm2,
                   h->status, cdg_rule_of(h));
  }
  return cudaGetLastError();
}

cudaError_t cdg_launch_fused(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st) {
  const int M = pick_M(h->m);
  if (h->dtype == CDGRAB_F32) {
    if (M == 4) return launch_fused_t<float, 4>(h, grads, count, st);
    if (M == 8) return launch_fused_t<float, 8>(h, grads, count, st);
    return launch_fused_t<float, 16>(h, grads, count, st);
  }
  if (M == 4) return launch_fused_t<__nv_bfloat16, 4>(h, grads, count, st);
  if (M == 8) return launch_fused_t<__nv_bfloat16, 8>(h, grads, count, st);
  return launch_fused_t<__nv_bfloat16, 16>(h, grads, count, st);
}

template <typename T, int M>
static cudaError_t launch_gram_fma_t(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    gram_fma_kernel<T, M><<<h->gram_chunks, 256, 0, st>>>((const T *)grads, h->r, h->m, h->d, h->partials);
  }
  {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    fma_combine_kernel<M><<<1, 6 * Tri<M>::NPAD, 0, st>>>(h->partials, h->gram_chunks, h->m, h->gram);
  }
  return cudaGetLastError();
}

cudaError_t cdg_launch_gram_fma(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const int M = pick_M(h->m);
  if (h->dtype == CDGRAB_F32) {
    if (M == 4) return launch_gram_fma_t<float, 4>(h, grads, st);
    if (M == 8) return launch_gram_fma_t<float, 8>(h, grads, st);
    return launch_gram_fma_t<float, 16>(h, grads, st);
  }
  if (M == 4) return launch_gram_fma_t<__nv_bfloat16, 4>(h, grads, st);
  if (M == 8) return launch_gram_fma_t<__nv_bfloat16, 8>(h, grads, st);
  return launch_gram_fma_t<__nv_bfloat16, 16>(h, grads, st);
}

// ------------------------------------------------------------------------------------
// TMA-pipelined pass 1 for m <= 16 and long rows.
//
// The thread-per-column Gram above keeps ~250 registers per thread, so only 8 warps fit on
// an SM and their own loads cannot cover the HBM latency.  Here the loads are taken off the
// compute warps: warp 8 (one lane) streams tiles of [2m rows x 256 columns] plus the
// matching 256 entries of r through a ring of shared-memory stages with bulk-tensor copies
// and mbarriers; the 256 compute threads each own one column of the tile, read its 2m
// values from shared memory (consecutive threads, consecutive words: no bank conflicts),
// form c = z1 - z2 and feed the same register-resident triangle of accumulators.
// Persistent CTAs take tiles blockIdx.x, blockIdx.x + gridDim.x, ...
// Waits are bounded; on expiry the CTA raises the time-out bit and stops consuming.
// ------------------------------------------------------------------------------------
#include <stdlib.h>

#include <type_traits>

#include "ptx.cuh"
#include "scan.cuh"

constexpr int kFtCols = 256;       // columns per tile
constexpr int kFtMaxStages = 8;
constexpr int kFtMaxGroups = 64;   // groups of the reduction tree over the CTAs
constexpr int kFtThreads = 2 * kFtCols + 32;   // two compute groups + the producer warp

template <typename T>
__device__ __forceinline__ float ft_widen(T v);
template <>
__device__ __forceinline__ float ft_widen<float>(float v) { return v; }
template <>
__device__ __forceinline__ float ft_widen<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <int I, int N, typename F>
__device__ __forceinline__ void static_for(F &&f) {
  if constexpr (I < N) {
    f(std::integral_constant<int, I>{});
    static_for<I + 1, N>(f);
  }
}

// The triangle of accumulators is shared out between two groups of 256 threads so that each
// thread needs about half the registers and twice as many warps fit: pair (a, b) belongs to
// group (a + b) & 1, the b-vector to group 1.  Local indices are compile-time constants.
template <int M>
struct Split {
  __host__ __device__ static constexpr int owner(int a, int b) { return (a + b) & 1; }
  __host__ __device__ static constexpr int count(int g) {
    int n = 0;
    for (int x = 0; x < M; ++x)
      for (int y = x; y < M; ++y) n += owner(x, y) == g;
    return n;
  }
  __host__ __device__ static constexpr int lidx(int a, int b) {
    int n = 0;
    for (int x = 0; x < M; ++x)
      for (int y = x; y < M; ++y) {
        if (x == a && y == b) return n;
        n += owner(x, y) == owner(a, b);
      }
    return n;
  }
  static constexpr int N0 = count(0);
  static constexpr int N1 = count(1) + M;       // odd pairs, then b
  static constexpr int NL = N0 > N1 ? N0 : N1;
  static constexpr int QL = (NL + 31) / 32;
  static constexpr int NLPAD = 32 * QL;
};

template <typename T, int M, int G>
__device__ __forceinline__ void ft_consume(const T *gt, const float *rt, int m, int col, float (&acc)[Split<M>::NLPAD]) {
  float c[M];
#pragma unroll
  for (int i = 0; i < M; ++i) {
    c[i] = 0.f;
    if (i < m)   // c = z1 - z2; columns past d were zero-filled by the copy
      c[i] = ft_widen<T>(gt[(size_t)i * kFtCols + col]) - ft_widen<T>(gt[(size_t)(m + i) * kFtCols + col]);
  }
  static_for<0, M>([&](auto A) {
    static_for<A.value, M>([&](auto B) {
      constexpr int a = A.value, b = B.value;
      if constexpr (Split<M>::owner(a, b) == G) {
        constexpr int l = Split<M>::lidx(a, b);
        acc[l] = fmaf(c[a], c[b], acc[l]);
      }
    });
  });
  if constexpr (G == 1) {
    const float rv = rt[col];
    static_for<0, M>([&](auto A) {
      constexpr int l = Split<M>::count(1) + A.value;
      acc[l] = fmaf(rv, c[A.value], acc[l]);
    });
  }
}

// Local entry (group, l) -> entry of the full triangle (row-major pairs a <= b, then b); -1: padding.
template <int M>
struct SplitMap {
  short v[2][Split<M>::NLPAD];
  constexpr SplitMap() : v{} {
    for (int g = 0; g < 2; ++g)
      for (int l = 0; l < Split<M>::NLPAD; ++l) v[g][l] = -1;
    int cnt[2] = {0, 0}, e = 0;
    for (int a = 0; a < M; ++a)
      for (int b = a; b < M; ++b) {
        const int g = Split<M>::owner(a, b);
        v[g][cnt[g]++] = (short)e++;
      }
    for (int a = 0; a < M; ++a) v[1][Split<M>::count(1) + a] = (short)(Tri<M>::NPAIR + a);
  }
};
template <int M>
__constant__ SplitMap<M> kSplitMap = SplitMap<M>();

// When enabled, the scalar part of the step runs inside this kernel (no scan launch).
using FtTail = CdgTail;

// Built with -DCDGRAB_STAMP (python -m paper_2302_00845_b200.build --stamp) every CTA of the
// TMA-fed kernel records %globaltimer at the phase boundaries of its last launch;
// cdgrab_debug_ft_stamps copies the table out ([CTA][slot], nanoseconds).  Off by default.
#ifdef CDGRAB_STAMP
constexpr int kFtStampSlots = 16;   // slot 10: kernel entry; slot 11: slot 9 of the launch before
__device__ unsigned long long ft_stamps[1024][kFtStampSlots];
__device__ __forceinline__ void ft_stamp(int slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  if (blockIdx.x < 1024) ft_stamps[blockIdx.x][slot] = t;
}
extern "C" int cdgrab_debug_ft_stamps(unsigned long long *host_out, int ctas) {
  if (ctas < 1 || ctas > 1024) return CDGRAB_ERR_INVALID;
  cudaDeviceSynchronize();
  return cudaMemcpyFromSymbol(host_out, ft_stamps, sizeof(unsigned long long) * kFtStampSlots * ctas) == cudaSuccess
             ? CDGRAB_OK : CDGRAB_ERR_CUDA;
}
#define FT_STAMP(cond, slot) do { if (cond) ft_stamp(slot); } while (0)
#else
#define FT_STAMP(cond, slot) do { } while (0)
#endif

// Fixed-order reduction tree over the CTAs, and what the whole-step mode needs.  The block
// partials are summed in two levels: CTAs form groups of `gsize`; the CTA that arrives last in
// its group (a counter per group) adds the group's partials in CTA order and publishes the group
// partial; a top counter counts finished groups.  The counters only ever grow: launch number
// `gen` (1, 2, ...) of a handle expects gen * (arrivals per launch), so nothing has to be reset
// and no CTA waits to take a ticket.
//   whole = 0: the CTA that finishes the last group combines the group partials, decides, leaves.
//   whole = 1: every CTA waits (bounded) until all groups are finished, combines the group
//              partials itself (same order everywhere, same bits), takes the same decisions, and
//              runs pass 2 over its own tiles in reverse: first the tiles still in its
//              shared-memory ring, then the ones most recently read (the likeliest to sit in L2).
//              CTAs wait on one another, so this mode is launched cooperatively.
struct FtTree {
  int whole;
  int gsize;                           // CTAs per group
  unsigned long long gen;              // launch number of this handle, from 1
  unsigned long long *group_ctr;       // [groups] arrivals, monotonic
  unsigned long long *top_ctr;         // [1] finished groups, monotonic
  double *group_partials;              // [groups][NACC]
  float *r;                            // whole-step and deferred-update modes: the running sum, updated in place
  // Deferred update: this launch first applies the update of the step BEFORE (whose signs are
  // known by now) to every tile of r it streams -- r <- r + sum_i s_i (z1_i - z2_i) over that
  // step's rows, which travel in the same stage -- stores the new r, and forms this step's Gram
  // matrix and b from it.  One read of r per step is saved and pass 2 of all but the last step of a
  // call needs no launch of its own.
  int fuse_prev;
  const int8_t *prev_signs;            // signs of the step before: prev_signs[i * prev_stride]
  int prev_stride;
};

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

template <typename T> struct FtAcc { typedef float type; };      // bf16 rows: fp32 adds, i ascending
template <> struct FtAcc<float> { typedef double type; };        // fp32 rows: one rounding of r per step

// pass 2 on one tile held in shared memory: r <- r + sum_i s_i (z1_i - z2_i), i ascending.
// All 2m values of the column are fetched before the first add, so the only serial part is the
// chain of m additions.
template <typename T, int M>
__device__ __forceinline__ float ft_update_tile(const T *gt, const float *rt, const float *ssh, int m, int col,
                                                long long gcol, long long d, float *__restrict__ r) {
  if (gcol >= d) return 0.f;
  float c[M];
#pragma unroll
  for (int i = 0; i < M; ++i) {
    c[i] = 0.f;
    if (i < m)
      c[i] = ssh[i] * (ft_widen<T>(gt[(size_t)i * kFtCols + col]) - ft_widen<T>(gt[(size_t)(m + i) * kFtCols + col]));
  }
  typename FtAcc<T>::type acc = (typename FtAcc<T>::type)rt[col];
#pragma unroll
  for (int i = 0; i < M; ++i)
    if (i < m) acc += (typename FtAcc<T>::type)c[i];
  const float out = (float)acc;
  r[gcol] = out;
  return out;
}

// FUSE: the launch also applies the update the step before left open (see FtTree); a separate
// instantiation, so that the plain pass 1 carries none of it.
template <typename T, int M, bool FUSE>
__global__ void __launch_bounds__(kFtThreads, 1)
gram_fma_tma_kernel(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_r,
                    const __grid_constant__ CUtensorMap tm_p, int m, long long d, int stages, int box_rows, int contiguous,
                    double *__restrict__ partials, int *__restrict__ status, const FtTail tail, const FtTree tree) {
  extern __shared__ uint8_t ft_smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kFtMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kFtMaxStages];
  __shared__ double red[16 * Split<M>::NLPAD];      // [warp][local entry]; afterwards the scan's arrays
  __shared__ float ssh[M];                          // signs of the step as +-1.0f (whole-step mode)
  __shared__ int flag_sh[3];                        // last of its group / finished the last group / wait ended well
  __shared__ int bad_sh;                            // a wait of this CTA has run out

#ifdef CDGRAB_STAMP
  if (threadIdx.x == 0 && blockIdx.x < 1024) ft_stamps[blockIdx.x][11] = ft_stamps[blockIdx.x][9];
  FT_STAMP(threadIdx.x == 0, 10);
#endif
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = warp >> 3;                       // 0, 1: compute groups; 2: producer
  const uint32_t base = (smem_u32(ft_smem_raw) + 127u) & ~127u;
  uint8_t *base_ptr = ft_smem_raw + (base - smem_u32(ft_smem_raw));
  const int nbox = (2 * m + box_rows - 1) / box_rows;             // row boxes per tile
  const uint32_t box_bytes = (uint32_t)box_rows * kFtCols * (uint32_t)sizeof(T);
  const uint32_t g_bytes = (uint32_t)nbox * box_bytes;            // rows past 2m are zero-filled
  const uint32_t r_bytes = kFtCols * (uint32_t)sizeof(float);
  // rows, then the r tile, then (deferred update) the rows of the step before
  const uint32_t stage_bytes = g_bytes + r_bytes + (FUSE ? g_bytes : 0u);
  const long long ntiles = (d + kFtCols - 1) / kFtCols;
  // tiles of this CTA: a contiguous range, or every gridDim.x-th tile
  const long long t_lo = contiguous ? ntiles * blockIdx.x / gridDim.x : blockIdx.x;
  const long long t_hi = contiguous ? ntiles * (blockIdx.x + 1) / gridDim.x : ntiles;
  const long long t_step = contiguous ? 1 : gridDim.x;
  const int n_iter = (int)((t_hi - t_lo + t_step - 1) / t_step);
  // whole-step mode: the last `keep` tiles of pass 1 stay in the ring for pass 2
  const int keep = tree.whole ? min(stages, n_iter) : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 16);  // one arrival per compute warp
    }
    mbar_init_fence();
    bad_sh = 0;
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_g) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_r) : "memory");
  }
  __syncthreads();
  FT_STAMP(threadIdx.x == 0, 0);
  cdg_grid_dep_wait();      // r is written by the launch before this one
  FT_STAMP(threadIdx.x == 0, 1);
  const long long deadline = clock64() + kCdgWaitCycles;
  if constexpr (FUSE) {     // the signs the launch before this one decided
    if (threadIdx.x < m) ssh[threadIdx.x] = (float)tree.prev_signs[(size_t)threadIdx.x * tree.prev_stride];
    __syncthreads();
  }

  float acc[Split<M>::NLPAD];
#pragma unroll
  for (int e = 0; e < Split<M>::NLPAD; ++e) acc[e] = 0.f;

  // what the scalar tail will need, fetched now by idle lanes of the producer warp
  int32_t pf_first = 0, pf_second = 0;
  double pf_rn2 = 0.0;
  bool prod_ok = true;                               // producer lane: no wait has run out so far
  if (group == 2) {
    if (tail.enabled && lane >= 1 && lane <= m) {
      pf_first = tail.perm_cur[(size_t)(lane - 1) * tail.n + 2 * tail.k];
      pf_second = tail.perm_cur[(size_t)(lane - 1) * tail.n + 2 * tail.k + 1];
    }
    if (tail.enabled && lane == 17) pf_rn2 = *tail.rnorm2;
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      int s = 0;
      uint32_t turn = 0;                       // how often the ring has wrapped
      for (int it = 0; it < n_iter; ++it) {
        if (turn > 0) ok = mbar_wait(smem_u32(&bar_empty[s]), (turn - 1) & 1, deadline);
        if (!ok) break;
        const long long tile = t_lo + (long long)it * t_step;
        const int col = (int)(tile * kFtCols);            // 256 elements: 16-byte aligned for both types
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t dst = base + s * stage_bytes;
        mbar_expect_tx(full, stage_bytes);
        for (int q = 0; q < nbox; ++q) tma_load_2d(dst + q * box_bytes, &tm_g, col, q * box_rows, full);
        tma_load_2d(dst + g_bytes, &tm_r, col, 0, full);
        if constexpr (FUSE)
          for (int q = 0; q < nbox; ++q) tma_load_2d(dst + g_bytes + r_bytes + q * box_bytes, &tm_p, col, q * box_rows, full);
        issued = it + 1;
        if (++s == stages) { s = 0; ++turn; }
      }
      if (!ok) {
        atomicOr(status, CDG_ST_TIMEOUT);
        bad_sh = 1;
        for (int it = max(0, issued - stages); it < issued; ++it)
          mbar_wait(smem_u32(&bar_full[it % stages]), (it / stages) & 1, clock64() + kCdgWaitCycles);
      }
      prod_ok = ok;
    }
  } else {
    const int col = threadIdx.x & (kFtCols - 1);
    bool ok = true;
    int s = 0;
    uint32_t parity = 0;
    for (int it = 0; it < n_iter && ok; ++it) {
      ok = mbar_wait(smem_u32(&bar_full[s]), parity, deadline);
      if (!ok) break;
      FT_STAMP(threadIdx.x == 0 && it == 0, 2);
      const T *gt = reinterpret_cast<const T *>(base_ptr + (size_t)s * stage_bytes);
      float *rt = reinterpret_cast<float *>(base_ptr + (size_t)s * stage_bytes + g_bytes);
      if (FUSE && group == 1) {
        // the update the step before left open, on this thread's column; the new value replaces
        // the old one in the stage so that b below is formed against it
        const T *pt = reinterpret_cast<const T *>(base_ptr + (size_t)s * stage_bytes + g_bytes + r_bytes);
        const long long gcol = (t_lo + (long long)it * t_step) * kFtCols + col;
        rt[col] = ft_update_tile<T, M>(pt, rt, ssh, m, col, gcol, d, tree.r);
      }
      if (group == 0) ft_consume<T, M, 0>(gt, rt, m, col, acc);
      else ft_consume<T, M, 1>(gt, rt, m, col, acc);
      __syncwarp();
      // this warp is done with the stage (a tile kept for pass 2 is released there instead)
      if (lane == 0 && it < n_iter - keep) mbar_arrive(smem_u32(&bar_empty[s]));
      if (++s == stages) { s = 0; parity ^= 1u; }
    }
    if (!ok && lane == 0) { atomicOr(status, CDG_ST_TIMEOUT); bad_sh = 1; }
    FT_STAMP(threadIdx.x == 0, 3);
    // warp totals of the local entries, as doubles
    warp_reduce_vec<Split<M>::NLPAD>(acc, lane);
#pragma unroll
    for (int q = 0; q < Split<M>::QL; ++q)
      red[warp * Split<M>::NLPAD + q + Split<M>::QL * lane] = (double)acc[q];
  }
  __syncthreads();
  // thread (g, l): add the 8 warps of group g in warp order, store under the triangle's entry
  if (threadIdx.x < 2 * Split<M>::NLPAD) {
    const int g = threadIdx.x / Split<M>::NLPAD, l = threadIdx.x % Split<M>::NLPAD;
    const int e = kSplitMap<M>.v[g][l];
    if (e >= 0) {
      double v = 0.0;
#pragma unroll
      for (int w = 0; w < 8; ++w) v += red[(g * 8 + w) * Split<M>::NLPAD + l];
      partials[(size_t)blockIdx.x * Tri<M>::NACC + e] = v;
    }
  }
  // a compute warp gave up on a tile: let the copies still under way land before the CTA can leave
  if (bad_sh && group == 2 && lane == 0 && prod_ok) {
    for (int it = max(0, n_iter - stages); it < n_iter; ++it)
      mbar_wait(smem_u32(&bar_full[it % stages]), (it / stages) & 1, clock64() + kCdgWaitCycles);
  }
  if (!tail.enabled) return;

  // ---- two-level tree over the CTAs (no CTA waits to take a ticket) ----
  constexpr int NACC = Tri<M>::NACC;
  const int grp = blockIdx.x / tree.gsize;
  const int ngroups = ((int)gridDim.x + tree.gsize - 1) / tree.gsize;
  const int gcount = min(tree.gsize, (int)gridDim.x - grp * tree.gsize);
  __threadfence();
  __syncthreads();                                   // red is free from here on
  if (threadIdx.x == 0) {
    const unsigned long long old = atomicAdd(tree.group_ctr + grp, 1ull);
    flag_sh[0] = (old + 1 == tree.gen * (unsigned long long)gcount);
    flag_sh[1] = 0;
    FT_STAMP(true, 4);
  }
  __syncthreads();
  if (flag_sh[0]) {
    // last of its group: the group's block partials in CTA order (all loads in flight first)
    __threadfence();
    if (threadIdx.x < NACC) {
      const double *src = partials + (size_t)grp * tree.gsize * NACC + threadIdx.x;
      double v = 0.0;
#pragma unroll 1
      for (int b0 = 0; b0 < gcount; b0 += 12) {
        double x[12];
#pragma unroll
        for (int q = 0; q < 12; ++q) x[q] = (b0 + q < gcount) ? __ldcg(src + (size_t)(b0 + q) * NACC) : 0.0;
#pragma unroll
        for (int q = 0; q < 12; ++q)
          if (b0 + q < gcount) v += x[q];
      }
      tree.group_partials[(size_t)grp * NACC + threadIdx.x] = v;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const unsigned long long old = atomicAdd(tree.top_ctr, 1ull);
      flag_sh[1] = (old + 1 == tree.gen * (unsigned long long)ngroups);
    }
    __syncthreads();
  }
  if (!tree.whole) {
    if (!flag_sh[1]) return;                         // only the CTA that finished the last group goes on
  } else {
    // every CTA needs the totals: bounded wait until all groups are finished
    if (threadIdx.x == 0) {
      const unsigned long long want = tree.gen * (unsigned long long)ngroups;
      bool ok = true;
      while (ld_acquire_u64(tree.top_ctr) < want) {
        if (clock64() > deadline) { ok = false; break; }
      }
      if (!ok) atomicOr(status, CDG_ST_TIMEOUT);
      flag_sh[2] = ok;
      FT_STAMP(true, 5);
    }
    __syncthreads();
    if (!flag_sh[2]) return;                         // nothing of this CTA is in flight at this point
  }
  __threadfence();
  FT_STAMP(threadIdx.x == 0, 12);
  const ScanSmem S = scan_smem(red, m);
  double *rn2_sh = S.g + (size_t)m * m;
  if (threadIdx.x < NACC) {
    const int e = threadIdx.x;
    double v = 0.0;
    for (int b0 = 0; b0 < ngroups; b0 += 16) {       // group partials in group order
      double x[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) x[q] = (b0 + q < ngroups) ? __ldcg(tree.group_partials + (size_t)(b0 + q) * NACC + e) : 0.0;
#pragma unroll
      for (int q = 0; q < 16; ++q)
        if (b0 + q < ngroups) v += x[q];
    }
    if (e < Tri<M>::NPAIR) {
      int a = 0, rem = e;
      while (rem >= M - a) { rem -= M - a; ++a; }
      const int b = a + rem;
      if (a < m && b < m) { S.g[a * m + b] = v; S.g[b * m + a] = v; }
    } else {
      const int a = e - Tri<M>::NPAIR;
      if (a < m) S.t[a] = v;
    }
  }
  if (group == 2) {
    if (lane >= 1 && lane <= m) { S.p[2 * (lane - 1)] = pf_first; S.p[2 * (lane - 1) + 1] = pf_second; }
    if (lane == 17) *rn2_sh = pf_rn2;
  }
  __syncthreads();
  FT_STAMP(threadIdx.x == 0, 13);
  // in whole-step mode every CTA takes the decisions, CTA 0 records them
  scan_decide_and_write(S, S.g, m, tail.n, tail.k, tail.perm_next, tail.signs, tail.margins, tail.rnorm2, status,
                        tail.rule, *rn2_sh, !tree.whole || blockIdx.x == 0);
  FT_STAMP(threadIdx.x == 0, 14);
  if (!tree.whole || bad_sh) return;                 // (after a failed pass 1 the sums mean nothing)
  if (threadIdx.x < m) ssh[threadIdx.x] = (float)S.s[threadIdx.x];
  __syncthreads();
  FT_STAMP(threadIdx.x == 0, 6);

  // ---- pass 2 over this CTA's tiles, newest first ----
  // Step j < keep takes the tile of pass-1 iteration n_iter - keep + j straight from the ring; step
  // j >= keep is load number n_iter + (j - keep) of the ring and brings tile n_iter - 1 - j back.
  // The compute groups take the tiles in turn; both release every stage so the ring's arrival
  // counts stay as in pass 1.
  if (group == 2) {
    if (lane == 0 && prod_ok) {
      int issued_lo = n_iter, issued = n_iter;
      bool ok = true;
      for (int j = keep; j < n_iter; ++j) {
        const int L = n_iter + (j - keep), s = L % stages;
        ok = mbar_wait(smem_u32(&bar_empty[s]), ((L / stages) - 1) & 1, deadline);
        if (!ok) break;
        const long long tile = t_lo + (long long)(n_iter - 1 - j) * t_step;
        const int col = (int)(tile * kFtCols);
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t dst = base + s * stage_bytes;
        mbar_expect_tx(full, stage_bytes);
        for (int q = 0; q < nbox; ++q) tma_load_2d(dst + q * box_bytes, &tm_g, col, q * box_rows, full);
        tma_load_2d(dst + g_bytes, &tm_r, col, 0, full);
        issued = L + 1;
      }
      if (!ok) {
        atomicOr(status, CDG_ST_TIMEOUT);
        for (int L = max(issued_lo, issued - stages); L < issued; ++L)
          mbar_wait(smem_u32(&bar_full[L % stages]), (L / stages) & 1, clock64() + kCdgWaitCycles);
      }
    }
  } else {
    const int col = threadIdx.x & (kFtCols - 1);
    bool ok = true;
    for (int j = 0; j < n_iter; ++j) {
      const int L = (j < keep) ? n_iter - keep + j : n_iter + (j - keep);
      const int it = (j < keep) ? n_iter - keep + j : n_iter - 1 - j;
      const int s = L % stages;
      FT_STAMP(threadIdx.x == 0 && j == keep, 7);
      if (j >= keep) ok = mbar_wait(smem_u32(&bar_full[s]), (L / stages) & 1, deadline);
      if (!ok) break;
      FT_STAMP(threadIdx.x == 0 && j == keep, 8);
      if ((j & 1) == group) {
        const T *gt = reinterpret_cast<const T *>(base_ptr + (size_t)s * stage_bytes);
        const float *rt = reinterpret_cast<const float *>(base_ptr + (size_t)s * stage_bytes + g_bytes);
        const long long tile = t_lo + (long long)it * t_step;
        ft_update_tile<T, M>(gt, rt, ssh, m, col, tile * kFtCols + col, d, tree.r);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_empty[s]));
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
    FT_STAMP(threadIdx.x == 0, 9);
  }
}

bool cdg_fma_tma_supported(int m, long long d, int dtype) {
  const int align = (dtype == CDGRAB_F32) ? 4 : 8;   // row pitch must be a multiple of 16 bytes
  return m <= 16 && d % align == 0 && d >= 65536 && cdg_tensor_map_encoder() != nullptr;
}

static bool ft_encode(CUtensorMap *map, const void *base, long long d, int rows, int box_rows, int elem_bytes) {
  typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                               const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  EncodeFn fn = (EncodeFn)cdg_tensor_map_encoder();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)kFtCols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int M>
static cudaError_t ft_set_smem(size_t smem) {
  const cudaError_t e = cdg_open_smem_limit(gram_fma_tma_kernel<T, M, false>);
  return e != cudaSuccess ? e : cdg_open_smem_limit(gram_fma_tma_kernel<T, M, true>);
}

int cdg_fma_tma_setup(cdgrab_ctx *h) {
  const size_t esz = h->dtype == CDGRAB_F32 ? 4 : 2;
  int box_rows = 8;   // few distinct rows per copy keeps the far-apart rows' pages local
  if (const char *e = getenv("CDGRAB_FT_BOXROWS")) {
    const int v = atoi(e);
    if (v >= 1 && v <= 32) box_rows = v;
  }
  h->fma_tma_boxrows = box_rows;
  h->fma_tma_contig = 1;
  h->fma_tma_fused = 1;      // CDGRAB_FT_FUSE_TAIL=0: separate combine and scan launches
  if (const char *e = getenv("CDGRAB_FT_FUSE_TAIL")) h->fma_tma_fused = atoi(e) ? 1 : 0;
  if (const char *e = getenv("CDGRAB_FT_CONTIG")) h->fma_tma_contig = atoi(e) ? 1 : 0;
  const int nbox = (2 * h->m + box_rows - 1) / box_rows;
  const size_t stage = (size_t)nbox * box_rows * kFtCols * esz + kFtCols * sizeof(float);
  int stages = (int)((200 * 1024) / stage);
  if (const char *e = getenv("CDGRAB_FT_STAGES")) {
    const int v = atoi(e);
    if (v >= 2 && v < stages) stages = v;
  }
  if (stages > kFtMaxStages) stages = kFtMaxStages;
  if (stages < 2) return CDGRAB_ERR_INVALID;
  h->fma_tma_stages = stages;
  h->fma_tma_smem = stages * stage + 128;
  // deferred update: a stage also carries the rows of the step before
  const size_t stage2 = stage + (size_t)nbox * box_rows * kFtCols * esz;
  int stages2 = (int)((200 * 1024) / stage2);
  if (stages2 > kFtMaxStages) stages2 = kFtMaxStages;
  h->fma_tma_stages2 = stages2;
  h->fma_tma_smem2 = stages2 * stage2 + 128;
  // CDGRAB_DEFER=1: cdgrab_step_many folds pass 2 of a step into pass 1 of the next one.  Off by
  // default: measured slower than two launches per step at every size tried (the update's loads and
  // adds land on the threads that also own b, and a stage holds two steps' rows, so the ring is half
  // as deep): 91 against 52 us per step at m = 16, d = 2^20 fp32; 773 against 436 us at m = 16,
  // d = 13.5 M bf16.
  h->fma_tma_defer = 0;
  if (const char *e = getenv("CDGRAB_DEFER")) h->fma_tma_defer = atoi(e) ? 1 : 0;
  if (stages2 < 2) h->fma_tma_defer = 0;
  const long long ntiles = (h->d + kFtCols - 1) / kFtCols;
  h->gram_chunks = (int)(ntiles < h->num_sms ? ntiles : h->num_sms);
  if (!ft_encode(&h->tm_fr, h->r, h->d, 1, 1, 4)) return CDGRAB_ERR_CUDA;
  const int M = pick_M(h->m);
  cudaError_t e;
  if (h->dtype == CDGRAB_F32)
    e = M == 4 ? ft_set_smem<float, 4>(h->fma_tma_smem) : M == 8 ? ft_set_smem<float, 8>(h->fma_tma_smem)
                                                                  : ft_set_smem<float, 16>(h->fma_tma_smem);
  else
    e = M == 4 ? ft_set_smem<__nv_bfloat16, 4>(h->fma_tma_smem)
               : M == 8 ? ft_set_smem<__nv_bfloat16, 8>(h->fma_tma_smem)
                        : ft_set_smem<__nv_bfloat16, 16>(h->fma_tma_smem);
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  // reduction tree over the CTAs: groups of 12 (more when the grid is wider than 64 groups of 12)
  h->ft_gsize = 12;
  while ((h->gram_chunks + h->ft_gsize - 1) / h->ft_gsize > kFtMaxGroups) ++h->ft_gsize;
  const size_t ctr_bytes = sizeof(unsigned long long) * (kFtMaxGroups + 1);
  const size_t gp_bytes = sizeof(double) * 152 * kFtMaxGroups;
  if (cdg_alloc(h, &h->ft_ctr, ctr_bytes) != cudaSuccess || cdg_alloc(h, &h->ft_group_partials, gp_bytes) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_NOMEM;
  }
  if (cudaMemset(h->ft_ctr, 0, ctr_bytes) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->ft_gen = 0;
  // CDGRAB_FT_WHOLE=1: pass 2 runs inside the pass-1 launch (measured slower than two chained
  // launches at every size tried, so off by default); needs a device that can keep the whole grid
  // resident (cooperative launch)
  h->fma_tma_whole = 0;
  if (const char *e = getenv("CDGRAB_FT_WHOLE")) h->fma_tma_whole = atoi(e) ? 1 : 0;
  h->ft_coop = 1;
  if (const char *e = getenv("CDGRAB_FT_COOP")) h->ft_coop = atoi(e) ? 1 : 0;

  int coop = 0;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h->device) != cudaSuccess || !coop) {
    cudaGetLastError();
    h->fma_tma_whole = 0;
  }
  h->fma_tma = 1;
  return CDGRAB_OK;
}

template <typename T, int M>
static cudaError_t launch_gram_fma_tma_t(cdgrab_ctx *h, const CUtensorMap &tm_g, const CUtensorMap *tm_prev,
                                         cudaStream_t st) {
  const FtTail tail = cdg_tail_of(h, h->fma_tma_fused);
  // the whole step in this launch unless something has to happen between the passes' launches
  const int whole = !tm_prev && h->fma_tma_whole && h->fma_tma_fused && !h->mean_out && !h->shard;
  FtTree tree;
  tree.whole = whole;
  tree.gsize = h->ft_gsize;
  tree.gen = h->fma_tma_fused ? ++h->ft_gen : 0;
  tree.group_ctr = h->ft_ctr;
  tree.top_ctr = h->ft_ctr + kFtMaxGroups;
  tree.group_partials = h->ft_group_partials;
  tree.r = h->r;
  tree.fuse_prev = tm_prev ? 1 : 0;
  tree.prev_signs = tm_prev ? h->signs + (h->k - 1) : nullptr;
  tree.prev_stride = h->n / 2;
  const int stages = tm_prev ? h->fma_tma_stages2 : h->fma_tma_stages;
  const size_t smem = tm_prev ? h->fma_tma_smem2 : h->fma_tma_smem;
  const CUtensorMap &tm_p = tm_prev ? *tm_prev : tm_g;
  h->ft_whole_launched = whole;
  {
    CdgProfScope ps(h, (whole || tm_prev) ? CDGRAB_K_FUSED : CDGRAB_K_GRAM, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(h->gram_chunks); cfg.blockDim = dim3(kFtThreads);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (whole && h->ft_coop) {   // its CTAs wait on one another: all of them must be resident
      at[na].id = cudaLaunchAttributeCooperative;
      at[na].val.cooperative = 1;
      ++na;
    }
    if (h->pdl && !(whole && h->ft_coop_no_pdl)) {
      at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[na].val.programmaticStreamSerializationAllowed = 1;
      ++na;
    }
    cfg.attrs = at; cfg.numAttrs = na;
    auto kernel = tm_prev ? gram_fma_tma_kernel<T, M, true> : gram_fma_tma_kernel<T, M, false>;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tm_g, h->tm_fr, tm_p, h->m, h->d, stages,
                                       h->fma_tma_boxrows, h->fma_tma_contig, h->partials, h->status, tail, tree);
    if (e != cudaSuccess && whole && h->ft_coop && na == 2) {
      // a driver that does not take both attributes together: cooperative alone from now on
      cudaGetLastError();
      h->ft_coop_no_pdl = 1;
      cfg.numAttrs = 1;
      e = cudaLaunchKernelEx(&cfg, kernel, tm_g, h->tm_fr, tm_p, h->m, h->d, stages,
                             h->fma_tma_boxrows, h->fma_tma_contig, h->partials, h->status, tail, tree);
    }
    if (e != cudaSuccess) return e;
  }
  if (!h->fma_tma_fused) {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    fma_combine_kernel<M><<<1, 6 * Tri<M>::NPAD, 0, st>>>(h->partials, h->gram_chunks, h->m, h->gram);
  }
  return cudaGetLastError();
}

// the tensor map over the 2m rows at `grads` (from the cache of the last few bases, or encoded now)
static const CUtensorMap *ft_map_of(cdgrab_ctx *h, const void *grads) {
  int slot = h->tm_fg.find(grads);
  if (slot < 0) {
    slot = h->tm_fg.victim();
    if (!ft_encode(&h->tm_fg.maps[slot][0], grads, h->d, 2 * h->m, h->fma_tma_boxrows, h->dtype == CDGRAB_F32 ? 4 : 2))
      return nullptr;
    h->tm_fg.commit(slot, grads);
  }
  return &h->tm_fg.maps[slot][0];
}

// grads_prev != NULL: the launch also applies the update of the step before, whose rows lie there
static cudaError_t ft_dispatch(cdgrab_ctx *h, const void *grads, const void *grads_prev, cudaStream_t st) {
  CUtensorMap prev_copy;
  const CUtensorMap *tp = nullptr;
  if (grads_prev) {
    const CUtensorMap *q = ft_map_of(h, grads_prev);
    if (!q) return cudaErrorInvalidValue;
    prev_copy = *q;                       // the cache entry may be replaced by the next look-up
    tp = &prev_copy;
  }
  const CUtensorMap *tg = ft_map_of(h, grads);
  if (!tg) return cudaErrorInvalidValue;
  const CUtensorMap &tm = *tg;
  const int M = pick_M(h->m);
  if (h->dtype == CDGRAB_F32) {
    if (M == 4) return launch_gram_fma_tma_t<float, 4>(h, tm, tp, st);
    if (M == 8) return launch_gram_fma_tma_t<float, 8>(h, tm, tp, st);
    return launch_gram_fma_tma_t<float, 16>(h, tm, tp, st);
  }
  if (M == 4) return launch_gram_fma_tma_t<__nv_bfloat16, 4>(h, tm, tp, st);
  if (M == 8) return launch_gram_fma_tma_t<__nv_bfloat16, 8>(h, tm, tp, st);
  return launch_gram_fma_tma_t<__nv_bfloat16, 16>(h, tm, tp, st);
}

cudaError_t cdg_launch_gram_fma_tma(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  return ft_dispatch(h, grads, nullptr, st);
}

cudaError_t cdg_launch_gram_fma_tma_deferred(cdgrab_ctx *h, const void *grads, const void *grads_prev, cudaStream_t st) {
  return ft_dispatch(h, grads, grads_prev, st);
}
