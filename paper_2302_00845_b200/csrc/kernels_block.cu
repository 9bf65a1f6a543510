// Pass 1 for more workers than the register-resident kernels hold (m > 16 outside the
// tensor-core path: fp32 gradients, bf16 with m > 64, odd row lengths): G = C^T C and b = C^T r
// over the step's pair differences c_i = z1_i - z2_i as a blocked product on the FMA pipe.
//
// The m rows are cut into blocks of 64; a CTA owns one pair of row blocks (I <= J) and a range
// of columns.  Per stage it forms the differences of 32 columns of both row blocks in shared
// memory (each input element is read once per block pair it belongs to), then every thread
// adds the products of an 8 x 8 patch of G (rows ty, ty+8, ... x columns tx, tx+8, ...) for its
// share of the stage's columns: 256 threads = 64 patches x 4 column phases.  fp32 partial sums
// are moved into an fp64 copy of the block in shared memory every 16384 columns (phase by
// phase, in a fixed order), so the length of an fp32 chain is bounded whatever d is; the CTA's
// fp64 block goes to global memory at the end and a second kernel adds the CTAs in index
// order.  Everything is deterministic.
#include "common.cuh"

namespace {

constexpr int kKT = 32;                    // columns per stage
constexpr int kKP = kKT + 1;               // row pitch in shared memory (conflict-free column reads)
constexpr int kFlushCols = 16384;          // columns between two moves of the fp32 sums into fp64

// BR rows per block: 64, or 32 when m <= 32 (a quarter of the products)
template <int BR>
struct BlockSmem {
  float ca[BR][kKP];
  float cb[BR][kKP];
  float rs[kKT];
  double acc64[BR * BR + BR];              // the block of G, then its b
};

// One CTA's work on the block pair (I, J).  256 threads = (BR/8)^2 patches of 8 x 8 entries x PH
// column phases; patch (ty, tx) holds rows ty, ty + BR/8, ... and columns tx, tx + BR/8, ...
template <typename T, int BR, bool DIAG>
__device__ __forceinline__ void gram_block_body(BlockSmem<BR> &S, const T *__restrict__ g,
                                                const float *__restrict__ r, int m, long long d, int I, int J,
                                                long long x_lo, long long x_hi, double *__restrict__ out) {
  constexpr int NP = BR / 8;               // patches per side
  constexpr int PH = 256 / (NP * NP);      // column phases
  constexpr int RW = BR / 8;               // rows each warp stages
  constexpr int ENT = BR * BR + BR;
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int phase = t / (NP * NP), ty = (t % (NP * NP)) / NP, tx = t % NP;
  for (int e = t; e < ENT; e += 256) S.acc64[e] = 0.0;

  float acc[8][8], bacc[DIAG ? 8 : 1];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (DIAG) bacc[i] = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  }
  auto flush = [&]() {
    // the column phases add their sums one after the other: a fixed order
    for (int s = 0; s < PH; ++s) {
      if (phase == s) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
#pragma unroll
          for (int j = 0; j < 8; ++j) S.acc64[(ty + NP * i) * BR + tx + NP * j] += (double)acc[i][j];
          if (DIAG && tx == 0) S.acc64[BR * BR + ty + NP * i] += (double)bacc[DIAG ? i : 0];
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (DIAG) bacc[i] = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
    }
  };

  const size_t slab = (size_t)m * (size_t)d;
  const float (*B)[kKP] = DIAG ? S.ca : S.cb;
  long long since = 0;
  // the differences of the next stage are fetched into registers while this one is multiplied
  float va[RW], vb[DIAG ? 1 : RW], vr = 0.f;
  auto fetch = [&](long long x0) {
    const long long x = x0 + lane;
    const bool inx = x < x_hi;
#pragma unroll
    for (int j = 0; j < RW; ++j) {
      const int rl = w + 8 * j;           // warp w takes rows w, w + 8, ... of the block, lane = column
      const int ra = I * BR + rl;
      va[j] = 0.f;
      if (inx && ra < m) {
        const size_t off = (size_t)ra * (size_t)d + (size_t)x;
        va[j] = cdg_ld(g + off) - cdg_ld(g + slab + off);   // c = z1 - z2
      }
      if (!DIAG) {
        const int rb = J * BR + rl;
        vb[j] = 0.f;
        if (inx && rb < m) {
          const size_t off = (size_t)rb * (size_t)d + (size_t)x;
          vb[j] = cdg_ld(g + off) - cdg_ld(g + slab + off);
        }
      }
    }
    if (DIAG) vr = (w == 0 && inx) ? r[x] : 0.f;
  };
  if (x_lo < x_hi) fetch(x_lo);
  __syncthreads();
  for (long long x0 = x_lo; x0 < x_hi; x0 += kKT) {
#pragma unroll
    for (int j = 0; j < RW; ++j) {
      S.ca[w + 8 * j][lane] = va[j];
      if (!DIAG) S.cb[w + 8 * j][lane] = vb[j];
    }
    if (DIAG && w == 0) S.rs[lane] = vr;
    if (x0 + kKT < x_hi) fetch(x0 + kKT);
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kKT / PH; ++kk) {
      const int k = phase + PH * kk;
      float a[8], b[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { a[i] = S.ca[ty + NP * i][k]; b[i] = B[tx + NP * i][k]; }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      if (DIAG && tx == 0) {
        const float rv = S.rs[k];
#pragma unroll
        for (int i = 0; i < 8; ++i) bacc[DIAG ? i : 0] = fmaf(rv, a[i], bacc[DIAG ? i : 0]);
      }
    }
    __syncthreads();
    since += kKT;
    if (since >= kFlushCols) { flush(); since = 0; }
  }
  flush();
  for (int e = t; e < ENT; e += 256) out[e] = S.acc64[e];
}

template <typename T, int BR>
__global__ void __launch_bounds__(256, 2)
gram_block_kernel(const T *__restrict__ g, const float *__restrict__ r, int m, long long d, int nblk,
                  long long cols_per_cta, double *__restrict__ partials) {
  extern __shared__ __align__(16) unsigned char bs_raw[];
  BlockSmem<BR> &S = *reinterpret_cast<BlockSmem<BR> *>(bs_raw);
  cdg_grid_dep_wait();            // r comes from the launch before this one
  int I = 0, rem = blockIdx.y;
  while (rem >= nblk - I) { rem -= nblk - I; ++I; }
  const int J = I + rem;
  const long long x_lo = (long long)blockIdx.x * cols_per_cta;
  const long long x_hi = (x_lo + cols_per_cta < d) ? x_lo + cols_per_cta : d;
  double *out = partials + ((size_t)blockIdx.x * gridDim.y + blockIdx.y) * (BR * BR + BR);
  if (I == J) gram_block_body<T, BR, true>(S, g, r, m, d, I, J, x_lo, x_hi, out);
  else gram_block_body<T, BR, false>(S, g, r, m, d, I, J, x_lo, x_hi, out);
}

// thread per (block pair, entry): add the CTAs in index order, scatter into the symmetric G
// (row-major [m][m]) and b ([m], stored after G)
__global__ void gram_block_combine_kernel(const double *__restrict__ partials, int ctas, int npairs, int nblk, int m,
                                          int kBR, double *__restrict__ gram) {
  cdg_grid_dep_wait();
  const int kEnt = kBR * kBR + kBR;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)npairs * kEnt) return;
  const int p = (int)(idx / kEnt), e = (int)(idx % kEnt);
  int I = 0, rem = p;
  while (rem >= nblk - I) { rem -= nblk - I; ++I; }
  const int J = I + rem;
  // entries outside the m x m matrix are never read: skip their sums
  int row, col = 0;
  if (e < kBR * kBR) { row = I * kBR + e / kBR; col = J * kBR + e % kBR; } else { row = I * kBR + (e - kBR * kBR); }
  if (row >= m || col >= m || (e >= kBR * kBR && I != J)) return;
  double v = 0.0;
  for (int c = 0; c < ctas; ++c) v += partials[((size_t)c * npairs + p) * kEnt + e];
  if (e < kBR * kBR) {
    gram[(size_t)row * m + col] = v;
    if (I != J) gram[(size_t)col * m + row] = v;
  } else {
    gram[(size_t)m * m + row] = v;
  }
}

}  // namespace

static int block_rows(const cdgrab_ctx *h) { return h->m <= 32 ? 32 : 64; }

// grid.x of the blocked Gram: about two CTAs per SM over all block pairs, at least one stage each
int cdg_block_ctas(const cdgrab_ctx *h) {
  const int br = block_rows(h), nblk = (h->m + br - 1) / br;
  const long long npairs = (long long)nblk * (nblk + 1) / 2;
  long long ctas = (2ll * h->num_sms + npairs - 1) / npairs;
  const long long maxc = (h->d + kKT - 1) / kKT;
  if (ctas > maxc) ctas = maxc;
  if (ctas < 1) ctas = 1;
  return (int)ctas;
}

size_t cdg_block_partials_bytes(const cdgrab_ctx *h) {
  const int br = block_rows(h), nblk = (h->m + br - 1) / br;
  return sizeof(double) * (size_t)(br * br + br) * (size_t)(nblk * (nblk + 1) / 2) * (size_t)cdg_block_ctas(h);
}

template <typename T, int BR>
static cudaError_t launch_gram_block_t(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const int nblk = (h->m + BR - 1) / BR;
  const int npairs = nblk * (nblk + 1) / 2;
  const int ctas = h->gram_chunks;
  long long cols = (h->d + ctas - 1) / ctas;
  cols = (cols + kKT - 1) / kKT * kKT;            // whole stages per CTA
  static CdgPerDevice attr_set;
  if (const cudaError_t e = cdg_raise_smem_limit(attr_set, h->device, gram_block_kernel<T, BR>, sizeof(BlockSmem<BR>));
      e != cudaSuccess)
    return e;
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    cdg_launch_dep(h, gram_block_kernel<T, BR>, dim3(ctas, npairs), dim3(256), sizeof(BlockSmem<BR>), st,
                   (const T *)grads, (const float *)h->r, h->m, h->d, nblk, cols, h->partials);
  }
  {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    const long long total = (long long)npairs * (BR * BR + BR);
    cdg_launch_dep(h, gram_block_combine_kernel, dim3((unsigned)((total + 127) / 128)), dim3(128), 0, st,
                   (const double *)h->partials, ctas, npairs, nblk, h->m, BR, h->gram);
  }
  return cudaGetLastError();
}

cudaError_t cdg_launch_gram_block(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const bool small = block_rows(h) == 32;
  if (h->dtype == CDGRAB_F32)
    return small ? launch_gram_block_t<float, 32>(h, grads, st) : launch_gram_block_t<float, 64>(h, grads, st);
  return small ? launch_gram_block_t<__nv_bfloat16, 32>(h, grads, st)
               : launch_gram_block_t<__nv_bfloat16, 64>(h, grads, st);
}
