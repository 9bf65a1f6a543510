// Parallel herding objective, Eq. (7) of the paper: the quantity PairBalance is meant to shrink,
//     max_k || sum_{j<=k} sum_i ( z[i][perm_i(j)] - zbar ) ||_inf ,   zbar = mean of all m*n vectors,
// evaluated on the device for m workers with n vectors of dimension d each.
//
// Every coordinate has its own running sum over the positions j, so the work is split into
// segments of consecutive positions: (1) raw sums of every segment, (2) per coordinate an
// exclusive prefix over the segments (which also yields the mean), (3) every segment walks its
// positions again from its starting value and tracks max |prefix|.  All sums are fp64 in a
// fixed order; the final maximum is exact, so the result does not depend on scheduling.
#include "common.cuh"

namespace {

struct HerdPlan {
  int nseg;        // segments of positions
  int seglen;      // positions per segment (the last one may be shorter)
};

HerdPlan herd_plan(int m, int n, long long d) {
  // about 160 gathered rows per thread: segments of 32 positions at m = 5, of one position at m >= 160
  const int want_len = m >= 160 ? 1 : 160 / m;
  long long nseg = (n + want_len - 1) / want_len;
  const long long cap = (8ll << 20) / d;          // at most 8 Mi (segment, coordinate) cells
  if (nseg > cap) nseg = cap;
  if (nseg < 1) nseg = 1;
  HerdPlan p;
  p.seglen = (int)((n + nseg - 1) / nseg);
  p.nseg = (n + p.seglen - 1) / p.seglen;
  return p;
}

// thread (segment, coordinate), coordinate fastest: sum_i z[i][perm_i(j)][x] over the segment
__global__ void herd_segment_sums(const float *__restrict__ z, const int32_t *__restrict__ perms, int m, int n,
                                  long long d, int nseg, int seglen, double *__restrict__ segsum) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= (long long)nseg * d) return;
  const int seg = (int)(g / d);
  const long long x = g % d;
  const int j0 = seg * seglen, j1 = min(n, j0 + seglen);
  double acc = 0.0;
  for (int j = j0; j < j1; ++j) {
    double step = 0.0;
    for (int i = 0; i < m; ++i) {
      const int32_t item = perms[(size_t)i * n + j];
      step += (double)z[((size_t)i * n + item) * (size_t)d + x];
    }
    acc += step;
  }
  segsum[g] = acc;
}

// thread per coordinate: exclusive prefix over the segments in place, mean into zbar
__global__ void herd_prefix(double *__restrict__ segsum, int nseg, long long d, double inv_count,
                            double *__restrict__ zbar) {
  const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= d) return;
  double run = 0.0;
  for (int s = 0; s < nseg; ++s) {
    const double v = segsum[(size_t)s * d + x];
    segsum[(size_t)s * d + x] = run;
    run += v;
  }
  zbar[x] = run * inv_count;
}

// Many segments (long sequences of short vectors): one block per coordinate.  Thread t adds a
// run of consecutive segments, thread 0 turns the 256 run totals into exclusive offsets in run
// order, then every thread writes the exclusive prefix of its run.  Fixed order throughout.
__global__ void __launch_bounds__(256)
herd_prefix_block(double *__restrict__ segsum, int nseg, long long d, double inv_count, double *__restrict__ zbar) {
  __shared__ double runs[256];
  const long long x = blockIdx.x;
  const int len = (nseg + 255) / 256;
  const int s0 = min(nseg, (int)threadIdx.x * len), s1 = min(nseg, s0 + len);
  double tot = 0.0;
  for (int s = s0; s < s1; ++s) tot += segsum[(size_t)s * d + x];
  runs[threadIdx.x] = tot;
  __syncthreads();
  if (threadIdx.x == 0) {
    double run = 0.0;
    for (int t = 0; t < 256; ++t) { const double v = runs[t]; runs[t] = run; run += v; }
    zbar[x] = run * inv_count;
  }
  __syncthreads();
  double run = runs[threadIdx.x];
  for (int s = s0; s < s1; ++s) {
    const double v = segsum[(size_t)s * d + x];
    segsum[(size_t)s * d + x] = run;
    run += v;
  }
}

// thread (segment, coordinate): walk the segment from its starting prefix, track max |prefix|
__global__ void herd_segment_max(const float *__restrict__ z, const int32_t *__restrict__ perms, int m, int n,
                                 long long d, int nseg, int seglen, const double *__restrict__ segsum,
                                 const double *__restrict__ zbar, unsigned long long *__restrict__ out_bits) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  double best = 0.0;
  if (g < (long long)nseg * d) {
    const int seg = (int)(g / d);
    const long long x = g % d;
    const int j0 = seg * seglen, j1 = min(n, j0 + seglen);
    const double mz = (double)m * zbar[x];
    double p = segsum[g] - (double)j0 * mz;       // centred prefix before position j0
    for (int j = j0; j < j1; ++j) {
      double step = 0.0;
      for (int i = 0; i < m; ++i) {
        const int32_t item = perms[(size_t)i * n + j];
        step += (double)z[((size_t)i * n + item) * (size_t)d + x];
      }
      p += step - mz;
      best = fmax(best, fabs(p));
    }
  }
  // block maximum, then one atomic per block; non-negative doubles order like their bit patterns
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) best = fmax(best, __shfl_down_sync(0xffffffffu, best, off));
  __shared__ double wmax[8];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    double b = wmax[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) b = fmax(b, wmax[w]);
    atomicMax(out_bits, (unsigned long long)__double_as_longlong(b));
  }
}

}  // namespace

extern "C" long long cdgrab_herding_workspace_bytes(int m, int n, long long d) {
  if (m < 1 || n < 1 || d < 1) return -1;
  const HerdPlan p = herd_plan(m, n, d);
  return (long long)sizeof(double) * ((long long)p.nseg * d + d);
}

extern "C" int cdgrab_herding_objective(const float *z_dev, const int32_t *perms_dev, int m, int n, long long d,
                                        void *workspace_dev, long long workspace_bytes, double *out_dev,
                                        void *stream) {
  if (!z_dev || !perms_dev || !workspace_dev || !out_dev || m < 1 || n < 1 || d < 1) return CDGRAB_ERR_INVALID;
  if (workspace_bytes < cdgrab_herding_workspace_bytes(m, n, d)) return CDGRAB_ERR_INVALID;
  if (((uintptr_t)workspace_dev & 7) != 0 || ((uintptr_t)out_dev & 7) != 0) return CDGRAB_ERR_INVALID;
  const HerdPlan p = herd_plan(m, n, d);
  cudaStream_t st = (cudaStream_t)stream;
  double *segsum = (double *)workspace_dev;
  double *zbar = segsum + (size_t)p.nseg * d;
  const long long cells = (long long)p.nseg * d;
  const unsigned gb = (unsigned)((cells + 255) / 256);
  if (cudaMemsetAsync(out_dev, 0, sizeof(double), st) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  herd_segment_sums<<<gb, 256, 0, st>>>(z_dev, perms_dev, m, n, d, p.nseg, p.seglen, segsum);
  if (p.nseg >= 512 && d <= 65536)
    herd_prefix_block<<<(unsigned)d, 256, 0, st>>>(segsum, p.nseg, d, 1.0 / ((double)m * n), zbar);
  else
    herd_prefix<<<(unsigned)((d + 127) / 128), 128, 0, st>>>(segsum, p.nseg, d, 1.0 / ((double)m * n), zbar);
  herd_segment_max<<<gb, 256, 0, st>>>(z_dev, perms_dev, m, n, d, p.nseg, p.seglen, segsum, zbar,
                                       (unsigned long long *)out_dev);
  if (cudaGetLastError() != cudaSuccess) return CDGRAB_ERR_CUDA;
  return CDGRAB_OK;
}
