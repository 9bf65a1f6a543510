// ID-GraB (PairBal): the uncoordinated baseline of the paper's experiments (Section 5) -- every
// worker i balances its own pair differences against its OWN running sum r_i, so the m
// decisions of a step do not depend on each other:
//     t_i = <r_i, c_i>,  s_i = +1 iff t_i < 0 (Algorithm 6),  r_i <- r_i + s_i c_i.
// pass 1: one (worker, column chunk) block grid of dot products with fixed-order fp64 combine,
// a decision kernel (signs, margins, permutation slots of Algorithm 7), pass 2: the m updates.
#include "common.cuh"

namespace {

// VEC consecutive columns of a row as floats: 16-byte loads (4 fp32 / 8 bf16), 8-byte (4 bf16), or scalar
template <typename T, int VEC>
__device__ __forceinline__ void ldrow(const T *p, float (&v)[VEC]) {
  if constexpr (VEC == 1) {
    v[0] = cdg_ld(p);
  } else if constexpr (sizeof(T) == 4) {
    static_assert(VEC == 4, "fp32 rows are read 4 columns at a time");
    const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  } else if constexpr (VEC == 4) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
    v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
  } else {
    static_assert(VEC == 8, "bf16 rows are read 8 or 4 columns at a time");
    const uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[2 * j] = __uint_as_float(w[j] << 16);
      v[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
}
// the worker's running sum (read and written by these kernels: plain loads)
template <int VEC>
__device__ __forceinline__ void ldr(const float *p, float (&v)[VEC]) {
  if constexpr (VEC == 1) {
    v[0] = p[0];
  } else {
#pragma unroll
    for (int q = 0; q < VEC / 4; ++q) {
      const float4 f = *reinterpret_cast<const float4 *>(p + 4 * q);
      v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
    }
  }
}

// Column groups a thread has in flight: 4 for 16-byte groups of fp32 rows, 2 for bf16 rows read 8
// columns at a time (their groups carry twice the columns, and with 4 of them the kernels need 128
// registers: two blocks per SM; measured 8 % (m = 32, d = 13.5 M) to 22 % (m = 64, d = 31 M) slower).
template <typename T, int VEC>
struct IndepUnroll { static constexpr int value = (sizeof(T) == 2 && VEC == 8) ? 2 : 4; };

// grid (chunks, m).  partials[(i * chunks + chunk) * 3 + {t, rr, cc}]
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
indep_dot_kernel(const T *__restrict__ g, const float *__restrict__ r, int m, long long d,
                 double *__restrict__ partials) {
  constexpr int kIndepUnroll = IndepUnroll<T, VEC>::value;
  cdg_grid_dep_wait();            // the sums were updated by the launch before this one
  const int i = blockIdx.y;
  const T *z1 = g + (size_t)i * (size_t)d, *z2 = g + ((size_t)m + i) * (size_t)d;
  const float *ri = r + (size_t)i * (size_t)d;
  float t = 0.f, rr = 0.f, cc = 0.f;
  double td = 0.0, rrd = 0.0, ccd = 0.0;
  const long long nvec = d / VEC;
  const long long stride = (long long)gridDim.x * blockDim.x;
  int since = 0;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride * kIndepUnroll) {
    float a[kIndepUnroll][VEC], b[kIndepUnroll][VEC], rv[kIndepUnroll][VEC];
#pragma unroll
    for (int u = 0; u < kIndepUnroll; ++u) {       // all loads of the batch before the first use
      const long long vv = v + u * stride;
      if (vv < nvec) {
        const size_t x = (size_t)vv * VEC;
        ldrow<T, VEC>(z1 + x, a[u]); ldrow<T, VEC>(z2 + x, b[u]); ldr<VEC>(ri + x, rv[u]);
      } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) { a[u][j] = 0.f; b[u][j] = 0.f; rv[u][j] = 0.f; }
      }
    }
#pragma unroll
    for (int u = 0; u < kIndepUnroll; ++u) {
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        const float c = a[u][j] - b[u][j];   // c = z1 - z2
        t = fmaf(rv[u][j], c, t); rr = fmaf(rv[u][j], rv[u][j], rr); cc = fmaf(c, c, cc);
      }
    }
    if (++since == 16) {             // keep the fp32 partial sums short
      td += t; rrd += rr; ccd += cc; t = rr = cc = 0.f; since = 0;
    }
  }
  td += t; rrd += rr; ccd += cc;
  __shared__ double red[8][3];
  double vals[3] = {td, rrd, ccd};
#pragma unroll
  for (int q = 0; q < 3; ++q) {
    double v = vals[q];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5][q] = v;
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    double v = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += red[w][threadIdx.x];
    partials[((size_t)i * gridDim.x + blockIdx.x) * 3 + threadIdx.x] = v;
  }
}

// thread per worker: combine in chunk order, decide, write signs / margins / permutation slots
__global__ void indep_decide_kernel(const double *__restrict__ partials, int chunks, int m, int n, int k,
                                    const int32_t *__restrict__ perm_cur, int32_t *__restrict__ perm_next,
                                    int8_t *__restrict__ signs, float *__restrict__ margins,
                                    int *__restrict__ status) {
  cdg_grid_dep_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= m) return;
  double t = 0.0, rr = 0.0, cc = 0.0;
  for (int c = 0; c < chunks; ++c) {
    const double *p = partials + ((size_t)i * chunks + c) * 3;
    t += p[0]; rr += p[1]; cc += p[2];
  }
  if (!(isfinite(t) && isfinite(rr) && isfinite(cc))) atomicOr(status, CDG_ST_NONFINITE);
  const int s = (t < 0.0) ? 1 : -1;   // Algorithm 6; a tie gives -1
  const size_t pos = (size_t)i * (n >> 1) + k;
  signs[pos] = (int8_t)s;
  const double den = rr * cc;
  margins[pos] = (den > 0.0) ? (float)(fabs(t) / sqrt(den)) : 0.f;
  const int32_t first = perm_cur[(size_t)i * n + 2 * k], second = perm_cur[(size_t)i * n + 2 * k + 1];
  perm_next[(size_t)i * n + k] = (s == 1) ? first : second;             // front slot
  perm_next[(size_t)i * n + (n - 1 - k)] = (s == 1) ? second : first;   // back slot
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256)
indep_update_kernel(const T *__restrict__ g, float *__restrict__ r, const int8_t *__restrict__ signs,
                    int sign_stride, int m, long long d) {
  constexpr int kIndepUnroll = IndepUnroll<T, VEC>::value;
  cdg_grid_dep_wait();            // the signs come from the launch before this one
  const int i = blockIdx.y;
  const float s = (float)signs[(size_t)i * sign_stride];
  const T *z1 = g + (size_t)i * (size_t)d, *z2 = g + ((size_t)m + i) * (size_t)d;
  float *ri = r + (size_t)i * (size_t)d;
  const long long nvec = d / VEC;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride * kIndepUnroll) {
    float a[kIndepUnroll][VEC], b[kIndepUnroll][VEC], rv[kIndepUnroll][VEC];
#pragma unroll
    for (int u = 0; u < kIndepUnroll; ++u) {
      const long long vv = v + u * stride;
      if (vv < nvec) {
        const size_t x = (size_t)vv * VEC;
        ldrow<T, VEC>(z1 + x, a[u]); ldrow<T, VEC>(z2 + x, b[u]); ldr<VEC>(ri + x, rv[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kIndepUnroll; ++u) {
      const long long vv = v + u * stride;
      if (vv < nvec) {
        float *dst = ri + (size_t)vv * VEC;
#pragma unroll
        for (int j = 0; j < VEC; ++j) rv[u][j] += s * (a[u][j] - b[u][j]);
        if constexpr (VEC == 1) {
          dst[0] = rv[u][0];
        } else {
#pragma unroll
          for (int q = 0; q < VEC / 4; ++q)
            *reinterpret_cast<float4 *>(dst + 4 * q) =
                make_float4(rv[u][4 * q], rv[u][4 * q + 1], rv[u][4 * q + 2], rv[u][4 * q + 3]);
        }
      }
    }
  }
}

template <typename T, int VEC>
cudaError_t launch_indep_t(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  dim3 grid(h->gram_chunks, h->m);
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    cdg_launch_dep(h, indep_dot_kernel<T, VEC>, grid, dim3(256), 0, st, (const T *)grads, h->r, h->m, h->d,
                   h->partials);
  }
  {
    CdgProfScope ps(h, CDGRAB_K_SCAN, st);
    cdg_launch_dep(h, indep_decide_kernel, dim3((h->m + 127) / 128), dim3(128), 0, st, h->partials, h->gram_chunks,
                   h->m, h->n, h->k, h->perm_cur, h->perm_next, h->signs, h->margins, h->status);
  }
  {
    CdgProfScope ps(h, CDGRAB_K_UPDATE, st);
    cdg_launch_dep(h, indep_update_kernel<T, VEC>, grid, dim3(256), 0, st, (const T *)grads, h->r, h->signs + h->k,
                   h->n / 2, h->m, h->d);
  }
  return cudaGetLastError();
}

}  // namespace

// column chunks per worker: enough blocks to fill the GPU, at most one per 1024 columns
int cdg_indep_chunks(const cdgrab_ctx *h) {
  long long want = (8ll * h->num_sms + h->m - 1) / h->m;
  const long long maxc = (h->d + 1023) / 1024;
  if (want > maxc) want = maxc;
  if (want < 1) want = 1;
  return (int)want;
}

cudaError_t cdg_launch_indep(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const bool v4 = (h->d % 4 == 0), v8 = (h->d % 8 == 0);
  if (h->dtype == CDGRAB_F32) return v4 ? launch_indep_t<float, 4>(h, grads, st) : launch_indep_t<float, 1>(h, grads, st);
  if (v8) return launch_indep_t<__nv_bfloat16, 8>(h, grads, st);
  return v4 ? launch_indep_t<__nv_bfloat16, 4>(h, grads, st) : launch_indep_t<__nv_bfloat16, 1>(h, grads, st);
}
