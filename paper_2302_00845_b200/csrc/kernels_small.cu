// The whole step in one CTA for many workers with short rows (17 <= m <= 128, the step's
// differences fit shared memory): the Gram form with every dot product taken in parallel.
//
// Applying Algorithm 6 worker by worker costs one block-wide reduction per worker, a chain of
// about half a microsecond each; with m = 100 workers of the paper's synthetic herding study
// (rows of 16 columns) that is 50 us per step for 13 KB of input.  Here the differences
// c_i = z1_i - z2_i are formed once into shared memory, G = C^T C (all m x m entries, one
// thread per entry, conflict-free because the row pitch is odd) and b = C^T r follow in
// parallel, the m decisions run as the register chain of the shared scan routine (tens of
// cycles per decision), and r <- r + sum_i s_i c_i closes the step.  `count` consecutive steps
// run in one launch with r in shared memory, rounded to fp32 once per step as every other path
// stores it.  Sums: fp32 over at most 64 columns at a time, moved into fp64; the update adds
// in worker order, in fp64 for fp32 rows (one rounding of r per step).  Deterministic.
#include "common.cuh"
#include "scan.cuh"

namespace {

constexpr int kSmallThreads = 1024;
constexpr int kSmallMaxM = 128;
constexpr size_t kSmallSmemBudget = 220 * 1024;

template <typename T>
__device__ __forceinline__ void small_ld4(const T *p, float (&v)[4]);
template <>
__device__ __forceinline__ void small_ld4<float>(const float *p, float (&v)[4]) {
  const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <>
__device__ __forceinline__ void small_ld4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[4]) {
  const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
  v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
  v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
}

template <typename T> struct SmallAcc { typedef float type; };      // bf16 rows: fp32 adds, i ascending
template <> struct SmallAcc<float> { typedef double type; };        // fp32 rows: one rounding of r per step

// shared memory: the scan's arrays and G ((4m + m*m) doubles), C [m][pitch] floats, r [d] floats
__host__ __device__ inline size_t small_smem_bytes(int m, long long d) {
  const size_t pitch = (size_t)d | 1;
  return scan_smem_bytes(m, true) + sizeof(float) * ((size_t)m * pitch + (size_t)d);
}

template <typename T>
__global__ void __launch_bounds__(kSmallThreads, 1)
gram_small_kernel(const T *__restrict__ g, int count, float *__restrict__ r_glob, int m, int d,
                  const CdgTail tail, int *__restrict__ status) {
  extern __shared__ double small_sh[];
  const ScanSmem S = scan_smem(small_sh, m);
  const int pitch = d | 1;                               // odd: rows start in different banks
  float *C = reinterpret_cast<float *>(small_sh + 4 * (size_t)m + (size_t)m * m);
  float *rsh = C + (size_t)m * pitch;
  const int tid = threadIdx.x, nth = blockDim.x;
  const size_t slab = (size_t)m * (size_t)d;
  const int nvec = d >> 2;
  cdg_grid_dep_wait();            // r and the current order may come from the launch before this one
  for (int x = tid; x < d; x += nth) rsh[x] = r_glob[x];

  for (int step = 0; step < count; ++step) {
    const int k = tail.k + step;
    const T *gs = g + (size_t)step * 2 * slab;
    __syncthreads();                                     // the step before is done with C, S and r
    scan_load_pairs(S, tail.perm_cur, m, tail.n, k);
    // differences into shared memory (Algorithm 2: z1 - z2)
    for (int e = tid; e < m * nvec; e += nth) {
      const int i = e / nvec, v = e - i * nvec;
      float a[4], b[4];
      small_ld4<T>(gs + (size_t)i * d + (size_t)v * 4, a);
      small_ld4<T>(gs + slab + (size_t)i * d + (size_t)v * 4, b);
      float *dst = C + (size_t)i * pitch + v * 4;
#pragma unroll
      for (int q = 0; q < 4; ++q) dst[q] = a[q] - b[q];
    }
    __syncthreads();
    // G[a][c] for all (a, c), and b[a] in column m of the same index space
    for (int e = tid; e < m * (m + 1); e += nth) {
      const int a = e / (m + 1), c = e - a * (m + 1);
      const float *pa = C + (size_t)a * pitch;
      const float *pc = (c < m) ? C + (size_t)c * pitch : rsh;
      double acc = 0.0;
      for (int x0 = 0; x0 < d; x0 += 64) {
        const int x1 = (x0 + 64 < d) ? x0 + 64 : d;
        float part = 0.f;
        for (int x = x0; x < x1; ++x) part = fmaf(pa[x], pc[x], part);
        acc += (double)part;
      }
      if (c < m) S.g[(size_t)a * m + c] = acc;
      else S.t[a] = acc;
    }
    __syncthreads();
    // the m decisions (Algorithm 6) and the permutation slots (Algorithm 7)
    scan_decide_and_write<4>(S, S.g, m, tail.n, k, tail.perm_next, tail.signs, tail.margins, tail.rnorm2, status,
                             tail.rule);
    // r <- r + sum_i s_i c_i, i ascending (S.s is visible: the routine synchronises after deciding)
    for (int x = tid; x < d; x += nth) {
      typename SmallAcc<T>::type acc = (typename SmallAcc<T>::type)rsh[x];
      for (int i = 0; i < m; ++i) acc += (typename SmallAcc<T>::type)((float)S.s[i] * C[(size_t)i * pitch + x]);
      rsh[x] = (float)acc;
    }
  }
  __syncthreads();
  for (int x = tid; x < d; x += nth) r_glob[x] = rsh[x];
}

}  // namespace

bool cdg_small_supported(int m, long long d, int dtype) {
  (void)dtype;
  return m > 16 && m <= kSmallMaxM && d % 4 == 0 && d >= 4 && d <= 4096 && small_smem_bytes(m, d) <= kSmallSmemBudget;
}

cudaError_t cdg_launch_small(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st) {
  static CdgPerDevice attr_f32, attr_bf16;
  const size_t smem = small_smem_bytes(h->m, h->d);
  cudaError_t e = h->dtype == CDGRAB_F32
                      ? cdg_raise_smem_limit(attr_f32, h->device, gram_small_kernel<float>, kSmallSmemBudget)
                      : cdg_raise_smem_limit(attr_bf16, h->device, gram_small_kernel<__nv_bfloat16>, kSmallSmemBudget);
  if (e != cudaSuccess) return e;
  CdgProfScope ps(h, CDGRAB_K_FUSED, st);
  if (h->dtype == CDGRAB_F32)
    e = cdg_launch_dep(h, gram_small_kernel<float>, dim3(1), dim3(kSmallThreads), smem, st, (const float *)grads, count,
                       h->r, h->m, (int)h->d, cdg_tail_of(h, 1), h->status);
  else
    e = cdg_launch_dep(h, gram_small_kernel<__nv_bfloat16>, dim3(1), dim3(kSmallThreads), smem, st,
                       (const __nv_bfloat16 *)grads, count, h->r, h->m, (int)h->d, cdg_tail_of(h, 1), h->status);
  return e != cudaSuccess ? e : cudaGetLastError();
}
