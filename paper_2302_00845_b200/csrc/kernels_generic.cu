// Generic two-pass path: works for every m, d and dtype the library accepts.
//
//   pass 1   gram_tile_kernel      G = C^T C and b = C^T r over the step's m pair
//                                  differences c_i = z1_i - z2_i, on the fp32 FMA pipe
//            gram_combine_kernel   fixed-order fp64 sum of the per-block partials
//   scan     scan_kernel           the m sequential sign decisions of Algorithm 6 in scalar
//                                  space, signs + next-permutation slots (Algorithm 7)
//   pass 2   update_kernel         r <- r + sum_i s_i c_i
//
// Inside a step r_{i-1} = r_0 + sum_{k<i} s_k c_k, hence
//   <r_{i-1}, c_i> = b_i + sum_{k<i} s_k G_ki,
// which is exact in real arithmetic and lets the d-sized work be done in two streaming
// passes instead of 2m dependent sweeps.
#include <stdlib.h>

#include <type_traits>

#include "common.cuh"
#include "scan.cuh"

// ------------------------------------------------------------------------------------
// pass 1 (generic): register-tiled Gram on FMA units
// grid = (chunks, tile pairs (I <= J)); each thread walks columns with a grid stride.
// ------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
gram_tile_kernel(const T *__restrict__ g, const float *__restrict__ r, int m, long long d,
                 int ntile, double *__restrict__ partials) {
  int I = 0, rem = blockIdx.y;
  while (rem >= ntile - I) { rem -= ntile - I; ++I; }
  const int J = I + rem;
  const bool diag = (I == J);

  float acc[CDG_TM][CDG_TM];
  float bacc[CDG_TM];
#pragma unroll
  for (int a = 0; a < CDG_TM; ++a) {
    bacc[a] = 0.f;
#pragma unroll
    for (int b = 0; b < CDG_TM; ++b) acc[a][b] = 0.f;
  }

  const long long stride = (long long)gridDim.x * blockDim.x;
  const size_t slab = (size_t)m * (size_t)d;
  for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < d; x += stride) {
    float cI[CDG_TM], cJ[CDG_TM];
#pragma unroll
    for (int a = 0; a < CDG_TM; ++a) {
      const int row = I * CDG_TM + a;
      cI[a] = 0.f;
      if (row < m) {
        const size_t off = (size_t)row * (size_t)d + (size_t)x;
        cI[a] = cdg_ld(g + off) - cdg_ld(g + slab + off);
      }
    }
    if (diag) {
      const float rx = r[x];
#pragma unroll
      for (int a = 0; a < CDG_TM; ++a) { cJ[a] = cI[a]; bacc[a] = fmaf(rx, cI[a], bacc[a]); }
    } else {
#pragma unroll
      for (int a = 0; a < CDG_TM; ++a) {
        const int row = J * CDG_TM + a;
        cJ[a] = 0.f;
        if (row < m) {
          const size_t off = (size_t)row * (size_t)d + (size_t)x;
          cJ[a] = cdg_ld(g + off) - cdg_ld(g + slab + off);
        }
      }
    }
#pragma unroll
    for (int a = 0; a < CDG_TM; ++a)
#pragma unroll
      for (int b = 0; b < CDG_TM; ++b) acc[a][b] = fmaf(cI[a], cJ[b], acc[a][b]);
  }

  // block reduction in fp64, fixed tree: lanes by shuffle, warps in index order
  __shared__ double red[8][CDG_TILE_ENTRIES];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int e = 0; e < CDG_TILE_ENTRIES; ++e) {
    double v = (e < CDG_TM * CDG_TM) ? (double)acc[e / CDG_TM][e % CDG_TM]
                                     : (double)bacc[e - CDG_TM * CDG_TM];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
    if (lane == 0) red[warp][e] = v;
  }
  __syncthreads();
  if (threadIdx.x < CDG_TILE_ENTRIES) {
    double v = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += red[w][threadIdx.x];
    partials[((size_t)blockIdx.x * gridDim.y + blockIdx.y) * CDG_TILE_ENTRIES + threadIdx.x] = v;
  }
}

// One thread per (tile pair, entry): sum the chunk partials in chunk order, scatter into the
// symmetric G (row-major [m][m]) and b ([m], stored after G).
__global__ void gram_combine_kernel(const double *__restrict__ partials, int chunks, int npairs,
                                    int ntile, int m, double *__restrict__ gram) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= npairs * CDG_TILE_ENTRIES) return;
  const int p = idx / CDG_TILE_ENTRIES, e = idx % CDG_TILE_ENTRIES;
  double v = 0.0;
  for (int c = 0; c < chunks; ++c) v += partials[((size_t)c * npairs + p) * CDG_TILE_ENTRIES + e];
  int I = 0, rem = p;
  while (rem >= ntile - I) { rem -= ntile - I; ++I; }
  const int J = I + rem;
  if (e < CDG_TM * CDG_TM) {
    const int row = I * CDG_TM + e / CDG_TM, col = J * CDG_TM + e % CDG_TM;
    if (row < m && col < m) {
      gram[(size_t)row * m + col] = v;
      if (I != J) gram[(size_t)col * m + row] = v;
    }
  } else if (I == J) {
    const int row = I * CDG_TM + (e - CDG_TM * CDG_TM);
    if (row < m) gram[(size_t)m * m + row] = v;
  }
}

// ------------------------------------------------------------------------------------
// scan: m sequential decisions in scalar space + permutation slots.  The block stages G, b
// and the current pairs in shared memory, warp 0 takes the decisions, the block writes out.
//   t_j starts as b_j; after worker i is decided every later t_j gains s_i G_ij, so when
//   worker j's turn comes t_j = <r_{j-1}, c_j> (summed in the order k = 0..j-1).
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
scan_kernel(const double *__restrict__ gram, int m, int n, int k,
            const int32_t *__restrict__ perm_cur, int32_t *__restrict__ perm_next,
            int8_t *__restrict__ signs, float *__restrict__ margins,
            double *__restrict__ rnorm2, int *__restrict__ status, int use_smem, const CdgRule rule) {
  extern __shared__ double sh[];
  cdg_grid_dep_wait();            // (G, b) come from the launch before this one
  const ScanSmem S = scan_smem(sh, m);
  const double *G = gram;
  for (int j = threadIdx.x; j < m; j += blockDim.x) S.t[j] = gram[(size_t)m * m + j];
  if (use_smem) {
    for (int e = threadIdx.x; e < m * m; e += blockDim.x) S.g[e] = gram[e];
    G = S.g;
  }
  scan_load_pairs(S, perm_cur, m, n, k);
  __syncthreads();
  scan_decide_and_write(S, G, m, n, k, perm_next, signs, margins, rnorm2, status, rule);
}

// ------------------------------------------------------------------------------------
// pass 2: r <- r + sum_i s_i (z1_i - z2_i), i ascending.  VEC columns per thread.
// AccT is double for fp32 inputs (one rounding of r per step), float for bf16 inputs.
// ------------------------------------------------------------------------------------
template <typename T, int VEC>
struct VecLoad;
template <>
struct VecLoad<float, 4> {
  static __device__ __forceinline__ void ld(const float *p, float (&v)[4]) {
    const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <>
struct VecLoad<float, 1> {
  static __device__ __forceinline__ void ld(const float *p, float (&v)[1]) { v[0] = __ldg(p); }
};
template <>
struct VecLoad<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&v)[8]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[2 * j] = __uint_as_float(w[j] << 16);
      v[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
};
// 256-bit loads (sm_100): one 32-byte request per row and thread
__device__ __forceinline__ void ld256(const void *p, uint32_t (&w)[8]) {
  asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
               : "l"(p));
}
// ... with the evict-first L2 priority: pass 2 is the last reader of a step's rows, so they may
// make room first (measured: pass 2 of the mid workload 30.3 -> 25.0 us on a slow box)
__device__ __forceinline__ void ld256_ef(const void *p, uint32_t (&w)[8]) {
  asm volatile("ld.global.nc.L2::evict_first.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
               : "l"(p));
}
template <>
struct VecLoad<__nv_bfloat16, 16> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&v)[16]) {
    uint32_t w[8];
    ld256(p, w);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      v[2 * j] = __uint_as_float(w[j] << 16);
      v[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ void ld_ef(const __nv_bfloat16 *p, float (&v)[16]) {
    uint32_t w[8];
    ld256_ef(p, w);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      v[2 * j] = __uint_as_float(w[j] << 16);
      v[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
};
template <>
struct VecLoad<float, 8> {
  static __device__ __forceinline__ void ld(const float *p, float (&v)[8]) {
    uint32_t w[8];
    ld256(p, w);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(w[j]);
  }
  static __device__ __forceinline__ void ld_ef(const float *p, float (&v)[8]) {
    uint32_t w[8];
    ld256_ef(p, w);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(w[j]);
  }
};
template <>
struct VecLoad<__nv_bfloat16, 1> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&v)[1]) {
    v[0] = __bfloat162float(*p);
  }
};

// MEAN: also write the parameter-server average of each gather buffer (Algorithm 4,
// "compute avg. gradient"): mean_out[q][x] = (1/m) sum_i grads[q][i][x], from the rows already
// in registers.
// EF: the rows are read with the evict-first L2 priority (256-bit loads only).
template <typename T, typename AccT, int VEC, bool SPLIT, bool MEAN, bool EF>
__global__ void __launch_bounds__(256)
update_kernel(const T *__restrict__ g, float *__restrict__ r, const int8_t *__restrict__ signs,
              int sign_stride, int m, long long d, __nv_bfloat16 *__restrict__ r_split,
              long long d_pad, float *__restrict__ mean_out) {
  extern __shared__ float ssh[];  // [m] signs as +-1.0f
  // The next launch in the stream (pass 1 of the next step) may be scheduled as this grid's blocks
  // leave; it waits for this grid's completion before it reads r.  (The pass-1 kernels do not
  // trigger early: pass 2's blocks would pile up on the SMs that finished first.)
  cdg_grid_dep_trigger();
  cdg_grid_dep_wait();            // the signs come from the launch before this one
  for (int i = threadIdx.x; i < m; i += blockDim.x) ssh[i] = (float)signs[(size_t)i * sign_stride];
  __syncthreads();
  const long long nvec = d / VEC;
  const size_t slab = (size_t)m * (size_t)d;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const size_t x = (size_t)v * VEC;
    AccT acc[VEC];
    float rv[VEC];
    if constexpr (VEC % 4 == 0) {
#pragma unroll
      for (int q = 0; q < VEC / 4; ++q) {
        const float4 f = *reinterpret_cast<const float4 *>(r + x + 4 * q);
        rv[4 * q] = f.x; rv[4 * q + 1] = f.y; rv[4 * q + 2] = f.z; rv[4 * q + 3] = f.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < VEC; ++j) rv[j] = r[x + j];
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] = (AccT)rv[j];
    float sa[MEAN ? VEC : 1], sb[MEAN ? VEC : 1];
    if constexpr (MEAN) {
#pragma unroll
      for (int j = 0; j < VEC; ++j) { sa[j] = 0.f; sb[j] = 0.f; }
    }
#pragma unroll 2
    for (int i = 0; i < m; ++i) {
      float a[VEC], b[VEC];
      if constexpr (EF) {        // nobody reads these rows again: they may leave L2 first
        VecLoad<T, VEC>::ld_ef(g + (size_t)i * (size_t)d + x, a);
        VecLoad<T, VEC>::ld_ef(g + slab + (size_t)i * (size_t)d + x, b);
      } else {
        VecLoad<T, VEC>::ld(g + (size_t)i * (size_t)d + x, a);
        VecLoad<T, VEC>::ld(g + slab + (size_t)i * (size_t)d + x, b);
      }
      const float s = ssh[i];
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[j] += (AccT)(s * (a[j] - b[j]));
      if constexpr (MEAN) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) { sa[j] += a[j]; sb[j] += b[j]; }
      }
    }
    if constexpr (MEAN) {
      const float inv_m = 1.f / (float)m;
      if constexpr (VEC % 4 == 0) {   // d is a multiple of VEC here: 16-byte aligned in both slabs
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q) {
          *reinterpret_cast<float4 *>(mean_out + x + 4 * q) =
              make_float4(sa[4 * q] * inv_m, sa[4 * q + 1] * inv_m, sa[4 * q + 2] * inv_m, sa[4 * q + 3] * inv_m);
          *reinterpret_cast<float4 *>(mean_out + (size_t)d + x + 4 * q) =
              make_float4(sb[4 * q] * inv_m, sb[4 * q + 1] * inv_m, sb[4 * q + 2] * inv_m, sb[4 * q + 3] * inv_m);
        }
      } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          mean_out[x + j] = sa[j] * inv_m;
          mean_out[(size_t)d + x + j] = sb[j] * inv_m;
        }
      }
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) rv[j] = (float)acc[j];
    if constexpr (VEC % 4 == 0) {
#pragma unroll
      for (int q = 0; q < VEC / 4; ++q)
        *reinterpret_cast<float4 *>(r + x + 4 * q) =
            make_float4(rv[4 * q], rv[4 * q + 1], rv[4 * q + 2], rv[4 * q + 3]);
    } else {
#pragma unroll
      for (int j = 0; j < VEC; ++j) r[x + j] = rv[j];
    }
    if constexpr (SPLIT) {
      // r = hi + mid + lo exactly (3 x 8 significand bits), consumed by the tensor-core pass
      __nv_bfloat16 hi[VEC], mid[VEC], lo[VEC];
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        hi[j] = __float2bfloat16_rn(rv[j]);
        const float r1 = rv[j] - __bfloat162float(hi[j]);
        mid[j] = __float2bfloat16_rn(r1);
        lo[j] = __float2bfloat16_rn(r1 - __bfloat162float(mid[j]));
      }
      if constexpr (VEC % 8 == 0) {
        // d_pad is a multiple of 64, x of 8: 16-byte aligned vector stores
#pragma unroll
        for (int q = 0; q < VEC / 8; ++q) {
          *reinterpret_cast<uint4 *>(r_split + x + 8 * q) = *reinterpret_cast<const uint4 *>(hi + 8 * q);
          *reinterpret_cast<uint4 *>(r_split + (size_t)d_pad + x + 8 * q) = *reinterpret_cast<const uint4 *>(mid + 8 * q);
          *reinterpret_cast<uint4 *>(r_split + 2 * (size_t)d_pad + x + 8 * q) = *reinterpret_cast<const uint4 *>(lo + 8 * q);
        }
      } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          r_split[x + j] = hi[j];
          r_split[(size_t)d_pad + x + j] = mid[j];
          r_split[2 * (size_t)d_pad + x + j] = lo[j];
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------
// per-example logistic-regression gradient for the current pair of every worker
// grid = (m, 2): block (i, q) handles item perm_cur[i][2k+q]
// ------------------------------------------------------------------------------------
template <bool VEC4>
__global__ void __launch_bounds__(256)
logreg_kernel(const float *__restrict__ X, const float *__restrict__ y, const float *__restrict__ w,
              const int32_t *__restrict__ perm_cur, int m, int n, long long d, int k,
              float *__restrict__ out) {
  cdg_grid_dep_wait();            // the buffer may still be read by the step launched before
  const int i = blockIdx.x, q = blockIdx.y;
  const int item = perm_cur[(size_t)i * n + 2 * k + q];
  const float *x = X + ((size_t)i * n + item) * (size_t)d;
  float part = 0.f;
  if constexpr (VEC4) {           // d % 4 == 0 and 16-byte aligned bases: the row stays in registers
    const long long nvec = d / 4;
    for (long long c = threadIdx.x; c < nvec; c += blockDim.x) {
      const float4 wv = __ldg(reinterpret_cast<const float4 *>(w) + c);
      const float4 xv = __ldg(reinterpret_cast<const float4 *>(x) + c);
      part = fmaf(wv.x, xv.x, part); part = fmaf(wv.y, xv.y, part);
      part = fmaf(wv.z, xv.z, part); part = fmaf(wv.w, xv.w, part);
    }
  } else {
    for (long long c = threadIdx.x; c < d; c += blockDim.x) part = fmaf(w[c], x[c], part);
  }
  __shared__ double red[8];
  __shared__ float coef;
  double v = (double)part;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double z = 0.0;
    for (int wi = 0; wi < 8; ++wi) z += red[wi];
    // sigma(z) - y without cancellation for y in {0,1}: sigma(z) - 1 = -sigma(-z)
    const float zf = (float)z;
    const float yv = y[(size_t)i * n + item];
    coef = (yv > 0.5f) ? -1.f / (1.f + expf(zf)) : 1.f / (1.f + expf(-zf));
  }
  __syncthreads();
  const float cf = coef;
  float *o = out + ((size_t)q * m + i) * (size_t)d;
  if constexpr (VEC4) {
    const long long nvec = d / 4;
    for (long long c = threadIdx.x; c < nvec; c += blockDim.x) {
      const float4 xv = __ldg(reinterpret_cast<const float4 *>(x) + c);   // second read: from L1/L2
      reinterpret_cast<float4 *>(o)[c] = make_float4(cf * xv.x, cf * xv.y, cf * xv.z, cf * xv.w);
    }
  } else {
    for (long long c = threadIdx.x; c < d; c += blockDim.x) o[c] = cf * x[c];
  }
}

// ------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------
cudaError_t cdg_launch_gram_generic(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  if (h->gram_block) return cdg_launch_gram_block(h, grads, st);
  const int ntile = (h->m + CDG_TM - 1) / CDG_TM;
  const int npairs = ntile * (ntile + 1) / 2;
  dim3 grid(h->gram_chunks, npairs);
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    if (h->dtype == CDGRAB_F32)
      gram_tile_kernel<float><<<grid, 256, 0, st>>>((const float *)grads, h->r, h->m, h->d, ntile,
                                                    h->partials);
    else
      gram_tile_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16 *)grads, h->r,
                                                            h->m, h->d, ntile, h->partials);
  }
  const int total = npairs * CDG_TILE_ENTRIES;
  {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    gram_combine_kernel<<<(total + 127) / 128, 128, 0, st>>>(h->partials, h->gram_chunks, npairs,
                                                             ntile, h->m, h->gram);
  }
  return cudaGetLastError();
}

cudaError_t cdg_launch_scan(cdgrab_ctx *h, cudaStream_t st) {
  const int m = h->m;
  const size_t small = scan_smem_bytes(m, false);
  const size_t with_g = scan_smem_bytes(m, true);
  const int use_smem = with_g <= 160 * 1024;
  const size_t smem = use_smem ? with_g : small;
  static CdgPerDevice attr_set;
  if (const cudaError_t e = cdg_raise_smem_limit(attr_set, h->device, scan_kernel, 160 * 1024); e != cudaSuccess)
    return e;
  {
    CdgProfScope ps(h, CDGRAB_K_SCAN, st);
    cdg_launch_dep(h, scan_kernel, dim3(1), dim3(256), smem, st, h->gram, m, h->n, h->k, h->perm_cur, h->perm_next,
                   h->signs, h->margins, h->rnorm2, h->status, use_smem, cdg_rule_of(h));
  }
  return cudaGetLastError();
}

template <typename T, typename AccT, int VEC, bool EF>
static void launch_update_t(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const long long nvec = h->d / VEC;
  long long blocks = (nvec + 255) / 256;
  const long long cap = (long long)h->num_sms * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const size_t smem = (size_t)h->m * sizeof(float);
  const int8_t *sg = h->signs + h->k;
  CdgProfScope ps(h, CDGRAB_K_UPDATE, st);
  if (h->mean_out) {
    if (h->r_split)
      cdg_launch_dep(h, update_kernel<T, AccT, VEC, true, true, false>, dim3((unsigned)blocks), dim3(256), smem, st,
                     (const T *)grads, h->r, sg, h->n / 2, h->m, h->d, h->r_split, h->d_pad, h->mean_out);
    else
      cdg_launch_dep(h, update_kernel<T, AccT, VEC, false, true, false>, dim3((unsigned)blocks), dim3(256), smem, st,
                     (const T *)grads, h->r, sg, h->n / 2, h->m, h->d, nullptr, 0, h->mean_out);
  } else if (h->r_split) {
    cdg_launch_dep(h, update_kernel<T, AccT, VEC, true, false, EF>, dim3((unsigned)blocks), dim3(256), smem, st,
                   (const T *)grads, h->r, sg, h->n / 2, h->m, h->d, h->r_split, h->d_pad, nullptr);
  } else {
    cdg_launch_dep(h, update_kernel<T, AccT, VEC, false, false, EF>, dim3((unsigned)blocks), dim3(256), smem, st,
                   (const T *)grads, h->r, sg, h->n / 2, h->m, h->d, nullptr, 0, nullptr);
  }
}

cudaError_t cdg_launch_update(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const bool al32 = ((uintptr_t)grads & 31) == 0;   // 256-bit loads need 32-byte aligned rows
  // with the average requested the two extra sums per column make the 256-bit variant
  // register-bound: the 128-bit one is faster then (measured +0.5 ms instead of +1.5 ms at m = 64)
  const bool wide = (h->mean_out == nullptr);
  const bool ef = h->upd_evict_first != 0;
  if (h->dtype == CDGRAB_F32) {
    if (al32 && h->d % 8 == 0 && wide) {
      if (ef) launch_update_t<float, double, 8, true>(h, grads, st);
      else launch_update_t<float, double, 8, false>(h, grads, st);
    } else if (h->d % 4 == 0) launch_update_t<float, double, 4, false>(h, grads, st);
    else launch_update_t<float, double, 1, false>(h, grads, st);
  } else {
    if (al32 && h->d % 16 == 0 && wide) {
      if (ef) launch_update_t<__nv_bfloat16, float, 16, true>(h, grads, st);
      else launch_update_t<__nv_bfloat16, float, 16, false>(h, grads, st);
    } else if (h->d % 8 == 0) launch_update_t<__nv_bfloat16, float, 8, false>(h, grads, st);
    else launch_update_t<__nv_bfloat16, float, 1, false>(h, grads, st);
  }
  return cudaGetLastError();
}

// stand-alone average of both gather buffers (used where pass 2 is part of a fused kernel)
template <typename T>
__global__ void mean_kernel(const T *__restrict__ g, int m, long long d, float *__restrict__ mean_out) {
  const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= 2 * d) return;
  const int q = (int)(x / d);
  const long long col = x % d;
  float acc = 0.f;
  for (int i = 0; i < m; ++i) acc += cdg_ld(g + ((size_t)q * m + i) * (size_t)d + col);
  mean_out[x] = acc * (1.f / (float)m);
}

cudaError_t cdg_launch_mean(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const unsigned blocks = (unsigned)((2 * h->d + 255) / 256);
  CdgProfScope ps(h, CDGRAB_K_UPDATE, st);
  if (h->dtype == CDGRAB_F32)
    mean_kernel<float><<<blocks, 256, 0, st>>>((const float *)grads, h->m, h->d, h->mean_out);
  else
    mean_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16 *)grads, h->m, h->d, h->mean_out);
  return cudaGetLastError();
}

// r -> its exact three-way bf16 split (after a state load on the tensor-core path)
__global__ void split_r_kernel(const float *__restrict__ r, long long d, long long d_pad,
                               __nv_bfloat16 *__restrict__ r_split) {
  const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= d) return;
  const float v = r[x];
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  r_split[x] = hi;
  r_split[(size_t)d_pad + x] = mid;
  r_split[2 * (size_t)d_pad + x] = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

cudaError_t cdg_launch_split_r(cdgrab_ctx *h, cudaStream_t st) {
  if (!h->r_split) return cudaSuccess;
  split_r_kernel<<<(unsigned)((h->d + 255) / 256), 256, 0, st>>>(h->r, h->d, h->d_pad, h->r_split);
  h->launches++;
  return cudaGetLastError();
}

cudaError_t cdg_launch_logreg(cdgrab_ctx *h, const float *X, const float *y, const float *w,
                              float *out, cudaStream_t st) {
  dim3 grid(h->m, 2);
  {
    CdgProfScope ps(h, CDGRAB_K_LOGREG, st);
    const bool vec4 = h->d % 4 == 0 && ((((uintptr_t)X) | ((uintptr_t)w) | ((uintptr_t)out)) & 15) == 0;
    if (vec4)
      cdg_launch_dep(h, logreg_kernel<true>, grid, dim3(256), 0, st, X, y, w, (const int32_t *)h->perm_cur, h->m,
                     h->n, h->d, h->k, out);
    else
      cdg_launch_dep(h, logreg_kernel<false>, grid, dim3(256), 0, st, X, y, w, (const int32_t *)h->perm_cur, h->m,
                     h->n, h->d, h->k, out);
  }
  return cudaGetLastError();
}
