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
#include "common.cuh"

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

// ------------------------------------------------------------------------------------
// Whole step in one CTA.  The thread count shrinks with M so the accumulators stay in
// registers: 1024 threads for M = 4, 512 for M = 8, 256 for M = 16.
// ------------------------------------------------------------------------------------
template <int M>
struct FusedCfg { static constexpr int THREADS = (M <= 4) ? 1024 : (M <= 8 ? 512 : 256); };

template <typename T, int M>
__global__ void __launch_bounds__(FusedCfg<M>::THREADS)
fused_step_kernel(const T *__restrict__ g, float *r, int m, int n, long long d, int k,
                  const int32_t *__restrict__ perm_cur, int32_t *__restrict__ perm_next,
                  int8_t *__restrict__ signs, float *__restrict__ margins,
                  double *__restrict__ rnorm2, int *__restrict__ status) {
  extern __shared__ double dsh[];
  constexpr int WARPS = FusedCfg<M>::THREADS / 32;
  double *red = dsh;                                  // [WARPS][NPAD]
  double *tot = red + WARPS * Tri<M>::NPAD;           // [NPAD]
  float *ssh = reinterpret_cast<float *>(tot + Tri<M>::NPAD);  // [M]

  float acc[Tri<M>::NPAD];
#pragma unroll
  for (int e = 0; e < Tri<M>::NPAD; ++e) acc[e] = 0.f;
  const long long nvec = d / 4;
  gram_accumulate<T, M>(g, r, m, d, threadIdx.x, blockDim.x, nvec, acc);
  const double v = block_reduce_acc<M, WARPS>(acc, red);
  if (threadIdx.x < Tri<M>::NACC) tot[threadIdx.x] = v;
  __syncthreads();

  if (threadIdx.x == 0) {
    // Algorithm 6 for i = 0..m-1 on t_i = b_i + sum_{k<i} s_k G_ki
    double t[M];
#pragma unroll
    for (int i = 0; i < M; ++i) t[i] = tot[Tri<M>::NPAIR + i];
    double rn2 = *rnorm2;
    bool bad = false;
    const int half = n >> 1;
#pragma unroll
    for (int i = 0; i < M; ++i) {
      if (i < m) {
        const double ti = t[i], gii = tot[Tri<M>::idx(i, i)];
        const int s = (ti < 0.0) ? 1 : -1;   // +1 iff ||r+c|| < ||r-c||; a tie gives -1
        bad |= !(isfinite(ti) && isfinite(gii));
        const double sd = (double)s;
#pragma unroll
        for (int j = i + 1; j < M; ++j) t[j] += sd * tot[Tri<M>::idx(i, j)];
        const size_t pos = (size_t)i * half + k;
        signs[pos] = (int8_t)s;
        const double den = rn2 * gii;
        margins[pos] = (den > 0.0) ? (float)(fabs(ti) / sqrt(den)) : 0.f;
        const int32_t first = perm_cur[(size_t)i * n + 2 * k];
        const int32_t second = perm_cur[(size_t)i * n + 2 * k + 1];
        perm_next[(size_t)i * n + k] = (s == 1) ? first : second;           // front slot
        perm_next[(size_t)i * n + (n - 1 - k)] = (s == 1) ? second : first;  // back slot
        rn2 += 2.0 * sd * ti + gii;
        if (rn2 < 0.0) rn2 = 0.0;
        ssh[i] = (float)s;
      }
    }
    *rnorm2 = rn2;
    if (bad) atomicOr(status, CDG_ST_NONFINITE);
  }
  __syncthreads();

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
}

// ------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------
static int pick_M(int m) { return m <= 4 ? 4 : (m <= 8 ? 8 : 16); }

bool cdg_fused_supported(int m, long long d, int dtype) {
  (void)dtype;
  return m <= 16 && d % 4 == 0;
}

template <typename T, int M>
static cudaError_t launch_fused_t(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const size_t smem = ((FusedCfg<M>::THREADS / 32) * Tri<M>::NPAD + Tri<M>::NPAD) * sizeof(double) +
                      M * sizeof(float);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(fused_step_kernel<T, M>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  {
    CdgProfScope ps(h, CDGRAB_K_FUSED, st);
    fused_step_kernel<T, M><<<1, FusedCfg<M>::THREADS, smem, st>>>(
        (const T *)grads, h->r, h->m, h->n, h->d, h->k, h->perm_cur, h->perm_next, h->signs,
        h->margins, h->rnorm2, h->status);
  }
  return cudaGetLastError();
}

cudaError_t cdg_launch_fused(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const int M = pick_M(h->m);
  if (h->dtype == CDGRAB_F32) {
    if (M == 4) return launch_fused_t<float, 4>(h, grads, st);
    if (M == 8) return launch_fused_t<float, 8>(h, grads, st);
    return launch_fused_t<float, 16>(h, grads, st);
  }
  if (M == 4) return launch_fused_t<__nv_bfloat16, 4>(h, grads, st);
  if (M == 8) return launch_fused_t<__nv_bfloat16, 8>(h, grads, st);
  return launch_fused_t<__nv_bfloat16, 16>(h, grads, st);
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
