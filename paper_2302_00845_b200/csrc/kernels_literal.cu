// The balancing step in its literal form, for short rows: Algorithm 6 applied worker by worker
// (Algorithm 7's inner loop as printed), one CTA, the running sum in registers.
//
// For i = 0..m-1 in order: c = z1_i - z2_i, t = <r, c>, s = +1 iff t < 0, r <- r + s c, and
// the two permutation slots of worker i.  Every decision needs a block-wide reduction, so the
// form only pays where a row is a few thousand columns at most (one CTA can hold r and a pair
// of rows in registers) -- there it replaces the Gram matrix, whose m(m+1)/2 products are more
// arithmetic than the m dot products they stand for, and it has no limit on m.
//
// Thread t owns the 4-column groups t, t + T (one or two of them: rows of up to 4096 columns);
// r lives in its registers as doubles for the whole launch (`count` consecutive steps; it is
// rounded to fp32 once per step, as a launch per step would store it); the rows of the next 2 to 8 workers are in flight
// while a worker is reduced (short rows leave registers for a deeper ring).  t and
// ||c||^2 are summed in fp64: lanes by a fixed butterfly, warps in index order through shared
// memory (two alternating slots, so one barrier per worker).  Deterministic.
#include "common.cuh"
#include "scan.cuh"

namespace {

constexpr int kLitMaxM = 1024;            // pairs of a step staged in shared memory

template <typename T>
__device__ __forceinline__ void lit_ld4(const T *p, float (&v)[4]);
template <>
__device__ __forceinline__ void lit_ld4<float>(const float *p, float (&v)[4]) {
  const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <>
__device__ __forceinline__ void lit_ld4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[4]) {
  const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
  v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
  v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
}

// CH: 4-column groups per thread; PF: workers whose rows are in flight ahead of the one being
// reduced (the sequence of workers runs on across the steps of the launch); MAXT: block size limit.
template <typename T, int CH, int PF, int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
literal_step_kernel(const T *__restrict__ g, int count, float *__restrict__ r_glob, int m, long long d,
                    const CdgTail tail, int *__restrict__ status) {
  __shared__ double red[2][32][2];         // [slot][warp][t, ||c||^2]
  __shared__ int32_t pairs[2 * kLitMaxM];
  // what the step's write-out needs about worker i, left there by the chain of decisions:
  // <r,c>, ||c||^2 (fp32 is enough for the reported margin) and the sign
  __shared__ double t_sh[kLitMaxM];
  __shared__ float cc_sh[kLitMaxM];
  __shared__ signed char s_sh[kLitMaxM];
  __shared__ double rn2_step;               // ||r||^2 at the start of the step
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nth = blockDim.x, nwarps = nth >> 5;
  const int nvec = (int)(d / 4);
  const size_t slab = (size_t)m * (size_t)d;
  cdg_grid_dep_wait();            // r and the current order may come from the launch before this one

  double r[CH][4];
#pragma unroll
  for (int j = 0; j < CH; ++j) {
    const int v = tid + j * nth;
#pragma unroll
    for (int q = 0; q < 4; ++q) r[j][q] = 0.0;
    if (v < nvec) {
      const float4 f = *reinterpret_cast<const float4 *>(r_glob + (size_t)v * 4);
      r[j][0] = f.x; r[j][1] = f.y; r[j][2] = f.z; r[j][3] = f.w;
    }
  }
  double rn2 = *tail.rnorm2;
  bool bad = false;
  int oob = 0, slot = 0;
  const int half = tail.n >> 1;
  const int total = count * m;             // (step, worker) pairs of this launch, in visiting order
  // lanes at and past the row's last column group hold zeros: the butterfly starts at the first
  // distance that still pairs two lanes with columns (16 for a full warp)
  int first_off = 16;
  while (first_off > 0 && first_off >= nvec) first_off >>= 1;

  // ring of PF row pairs; pw = the next (step, worker) to fetch
  float a[PF][CH][4], b[PF][CH][4];
  const T *prow = g;                        // row of slab 0 of the next worker to fetch
  int pi = 0;
  auto fetch = [&](float (&fa)[CH][4], float (&fb)[CH][4]) {
#pragma unroll
    for (int j = 0; j < CH; ++j) {
      const int v = tid + j * nth;
      if (v < nvec) {
        lit_ld4<T>(prow + (size_t)v * 4, fa[j]);
        lit_ld4<T>(prow + slab + (size_t)v * 4, fb[j]);
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) { fa[j][q] = 0.f; fb[j][q] = 0.f; }
      }
    }
    prow += d;
    if (++pi == m) { pi = 0; prow += slab; }   // on to slab 0 of the next step
  };
#pragma unroll
  for (int u = 0; u < PF; ++u)
    if (u < total) fetch(a[u], b[u]);

  int i = 0, k = tail.k;
  for (int w0 = 0; w0 < total; w0 += PF) {
#pragma unroll
    for (int u = 0; u < PF; ++u) {
      if (w0 + u < total) {
        if (i == 0) {
          __syncthreads();                 // the write-out of the step before is over
          for (int j = tid; j < 2 * m; j += nth) pairs[j] = tail.perm_cur[(size_t)(j >> 1) * tail.n + 2 * k + (j & 1)];
          if (tid == 0) rn2_step = rn2;
        }
        float c[CH][4];
#pragma unroll
        for (int j = 0; j < CH; ++j)
#pragma unroll
          for (int q = 0; q < 4; ++q) c[j][q] = a[u][j][q] - b[u][j][q];      // Algorithm 2: z1 - z2
        if (w0 + u + PF < total) fetch(a[u], b[u]);                            // the slot is free: PF workers ahead
        // <r, c> in fp64 (it takes the decision); ||c||^2 only feeds the reported margin and the
        // tracked norm, so its lane sums stay in fp32 (the fp64 pipe is the chain's slow part)
        // (the chain from one decision to the next runs through these sums: two short fp64 chains
        // per group instead of one long one, and only as many butterfly rounds as lanes hold columns)
        double t = 0.0;
        float ccf = 0.f;
#pragma unroll
        for (int j = 0; j < CH; ++j) {
          const double t0 = fma(r[j][1], (double)c[j][1], r[j][0] * (double)c[j][0]);
          const double t1 = fma(r[j][3], (double)c[j][3], r[j][2] * (double)c[j][2]);
          t += t0 + t1;
#pragma unroll
          for (int q = 0; q < 4; ++q) ccf = fmaf(c[j][q], c[j][q], ccf);
        }
        for (int off = first_off; off > 0; off >>= 1) {
          t += __shfl_xor_sync(0xffffffffu, t, off);
          ccf += __shfl_xor_sync(0xffffffffu, ccf, off);
        }
        double cc = (double)ccf;
        if (nwarps > 1) {
          if (lane == 0) { red[slot][warp][0] = t; red[slot][warp][1] = cc; }
          __syncthreads();
          t = 0.0; cc = 0.0;
          for (int w = 0; w < nwarps; ++w) { t += red[slot][w][0]; cc += red[slot][w][1]; }
          slot ^= 1;
        }
        // Algorithm 6: +1 iff ||r + c|| < ||r - c||  <=>  <r,c> < 0 (or the randomized rule)
        const int s = cdg_decide(tail.rule, i, t, oob);
        bad |= !(isfinite(t) && isfinite(cc));
        const double sd = (double)s;
#pragma unroll
        for (int j = 0; j < CH; ++j)
#pragma unroll
          for (int q = 0; q < 4; ++q) r[j][q] += sd * (double)c[j][q];
        if (tid == 0) { t_sh[i] = t; cc_sh[i] = (float)cc; s_sh[i] = (signed char)s; }
        rn2 += 2.0 * sd * t + cc;
        if (rn2 < 0.0) rn2 = 0.0;
        if (++i == m) {
          // end of a step: r takes the fp32 value a launch per step would have stored, so that a
          // staged call gives the bits of the same steps taken one by one
          i = 0;
#pragma unroll
          for (int j = 0; j < CH; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) r[j][q] = (double)(float)r[j][q];
          // The step's write-out, off the chain of decisions and by all threads: signs, margins
          // |t| / (||r|| ||c||) with ||r||^2 rebuilt worker by worker from the step's start, and
          // Algorithm 7's slots: the item that received +1 to the front slot k, the other to n-1-k.
          __syncthreads();
          if (CDG_IDX_OK(k >= 0 && k < half, status)) {
            for (int w = tid; w < m; w += nth) {
              const int sw = s_sh[w];
              const size_t pos = (size_t)w * half + k;
              tail.signs[pos] = (int8_t)sw;
              const int32_t first = pairs[2 * w], second = pairs[2 * w + 1];
              tail.perm_next[(size_t)w * tail.n + k] = (sw == 1) ? first : second;
              tail.perm_next[(size_t)w * tail.n + (tail.n - 1 - k)] = (sw == 1) ? second : first;
            }
            if (warp == 0) {
              // ||r||^2 seen by worker w = start + sum_{v<w} (2 s_v t_v + ||c_v||^2): a running sum, 32 workers at a time
              double base = rn2_step;
              for (int w0 = 0; w0 < m; w0 += 32) {
                const int w = w0 + lane;
                const double inc = (w < m) ? 2.0 * (double)s_sh[w] * t_sh[w] + (double)cc_sh[w] : 0.0;
                double pre = inc;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                  const double up = __shfl_up_sync(0xffffffffu, pre, off);
                  if (lane >= off) pre += up;
                }
                if (w < m) {
                  const double before = base + (pre - inc);
                  const float den = sqrtf(before > 0.0 ? (float)before : 0.f) * sqrtf(cc_sh[w]);
                  tail.margins[(size_t)w * half + k] = (den > 0.f) ? (float)fabs(t_sh[w]) / den : 0.f;
                }
                base += __shfl_sync(0xffffffffu, pre, 31);
              }
            }
          }
          ++k;
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < CH; ++j) {
    const int v = tid + j * nth;
    if (v < nvec)
      *reinterpret_cast<float4 *>(r_glob + (size_t)v * 4) =
          make_float4((float)r[j][0], (float)r[j][1], (float)r[j][2], (float)r[j][3]);
  }
  if (tid == 0) {
    *tail.rnorm2 = rn2;
    if (bad) atomicOr(status, CDG_ST_NONFINITE);
    if (oob) atomicAdd(tail.rule.oob, (unsigned long long)oob);
  }
}

template <typename T, int CH, int PF, int MAXT>
cudaError_t lit_launch(cdgrab_ctx *h, const void *grads, int count, int threads, cudaStream_t st) {
  return cdg_launch_dep(h, literal_step_kernel<T, CH, PF, MAXT>, dim3(1), dim3(threads), 0, st, (const T *)grads, count,
                        h->r, h->m, h->d, cdg_tail_of(h, 1), h->status);
}

template <typename T>
cudaError_t lit_dispatch(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st) {
  const int nvec = (int)(h->d / 4);
  auto round32 = [](int x) { return x < 32 ? 32 : (x + 31) & ~31; };
  // the shorter the rows, the fewer threads and the more registers for rows in flight
  if (nvec <= 256) return lit_launch<T, 1, 8, 256>(h, grads, count, round32(nvec), st);
  if (nvec <= 512) return lit_launch<T, 1, 4, 512>(h, grads, count, round32(nvec), st);
  return lit_launch<T, 2, 2, 512>(h, grads, count, round32((nvec + 1) / 2), st);
}

}  // namespace

// rows that one CTA of 512 threads holds with at most two 4-column groups per thread
bool cdg_literal_supported(int m, long long d, int dtype) {
  (void)dtype;
  return m >= 1 && m <= kLitMaxM && d % 4 == 0 && d >= 4 && d <= 4096;
}

cudaError_t cdg_launch_literal(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st) {
  CdgProfScope ps(h, CDGRAB_K_FUSED, st);
  const cudaError_t e = h->dtype == CDGRAB_F32 ? lit_dispatch<float>(h, grads, count, st)
                                               : lit_dispatch<__nv_bfloat16>(h, grads, count, st);
  return e != cudaSuccess ? e : cudaGetLastError();
}
