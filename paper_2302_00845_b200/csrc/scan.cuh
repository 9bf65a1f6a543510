// The scalar part of a balancing step, shared by the stand-alone scan kernel and by Gram
// kernels that finish the step themselves: m sequential sign decisions (Algorithm 6) on
//   t_i = b_i + sum_{k<i} s_k G_ki
// and the two permutation slots per worker (Algorithm 7).  Block-wide routines: every thread
// of the block must call them; shared memory is handed in by the caller.
#pragma once

#include "common.cuh"

// Which balance rule decides the signs.  Greedy (Algorithm 6): +1 iff <r,c> < 0.
// Randomized (Algorithm 2's subroutine with the bound w of Algorithm 5): p = 1/2 - <r,c>/(2w),
// +1 iff u_i < p with u_i the caller's uniform draw for worker i; positions with |<r,c>| > w
// (where Algorithm 5 would stop) are counted in *oob.
struct CdgRule {
  int randomized;
  const float *u;             // [m] uniforms in [0,1), device; NULL: drawn from (seed, epoch, k, i)
  double w;
  unsigned long long *oob;    // device counter
  unsigned long long seed;    // seeded draws: Philox4x32-10 keyed by the seed, counter (i, k, epoch, 0)
  unsigned epoch, k;
};

// Philox4x32-10 (Salmon et al., SC 2011): ten rounds of
//   (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)),
// the key advancing by the Weyl constants after each round.  Returns the first output word.
__host__ __device__ inline uint32_t cdg_philox4x32_10_first(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                            uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const unsigned long long p0 = 0xD2511F53ull * c0, p1 = 0xCD9E8D57ull * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1; c3 = (uint32_t)p0; c0 = n0; c2 = n2;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}
// the draw of worker i at pair index k of an epoch: top 24 bits of the word, times 2^-24
__host__ __device__ inline float cdg_seeded_uniform(unsigned long long seed, unsigned epoch, unsigned k, unsigned i) {
  const uint32_t x = cdg_philox4x32_10_first(i, k, epoch, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
  return (float)(x >> 8) * (1.0f / 16777216.0f);
}

__device__ __forceinline__ int cdg_decide(const CdgRule &rule, int i, double ti, int &oob_local) {
  if (!rule.randomized) return (ti < 0.0) ? 1 : -1;   // a tie gives -1
  const double p = 0.5 - ti / (2.0 * rule.w);
  if (fabs(ti) > rule.w) ++oob_local;
  const float u = rule.u ? rule.u[i] : cdg_seeded_uniform(rule.seed, rule.epoch, rule.k, (unsigned)i);
  return ((double)u < p) ? 1 : -1;
}

inline CdgRule cdg_rule_of(const cdgrab_ctx *h) {
  CdgRule r;
  r.randomized = h->rule_randomized;
  r.u = h->rule_u;
  r.w = h->rule_w;
  r.oob = h->oob;
  r.seed = h->rule_seed;
  r.epoch = h->rule_epoch;
  r.k = (unsigned)h->k;
  return r;
}

// What a pass-1 kernel needs to finish the step itself: the block that takes the last ticket
// runs the scalar part (no block ever waits for another).
struct CdgTail {
  int enabled;
  int n, k;
  unsigned *ticket;          // zero between launches
  const int32_t *perm_cur;
  int32_t *perm_next;
  int8_t *signs;
  float *margins;
  double *rnorm2;
  CdgRule rule;
};

inline CdgTail cdg_tail_of(const cdgrab_ctx *h, int enabled) {
  CdgTail t;
  t.enabled = enabled;
  t.n = h->n; t.k = h->k;
  t.ticket = h->ticket;
  t.perm_cur = h->perm_cur; t.perm_next = h->perm_next;
  t.signs = h->signs; t.margins = h->margins; t.rnorm2 = h->rnorm2;
  t.rule = cdg_rule_of(h);
  return t;
}

struct ScanSmem {
  double *t;     // [m]  starts as b; entry i is <r_{i-1}, c_i> once worker i is decided
  double *rn;    // [m]  ||r||^2 seen by worker i
  int *s;        // [m]  signs
  int *p;        // [2m] the current pair of every worker
  double *g;     // [m][m] optional copy of G
};

// (4m + m*m) doubles
__device__ __forceinline__ ScanSmem scan_smem(double *sh, int m) {
  ScanSmem S;
  S.t = sh;
  S.rn = sh + m;
  S.s = reinterpret_cast<int *>(sh + 2 * m);
  S.p = S.s + m;
  S.g = sh + 4 * m;
  return S;
}
__host__ __device__ inline size_t scan_smem_bytes(int m, bool with_g) {
  return ((size_t)4 * m + (with_g ? (size_t)m * m : 0)) * sizeof(double);
}

__device__ __forceinline__ void scan_load_pairs(const ScanSmem &S, const int32_t *__restrict__ perm_cur, int m,
                                                int n, int k) {
  for (int j = threadIdx.x; j < m; j += blockDim.x) {
    S.p[2 * j] = perm_cur[(size_t)j * n + 2 * k];
    S.p[2 * j + 1] = perm_cur[(size_t)j * n + 2 * k + 1];
  }
}

// The chain of decisions in registers for m <= 32 Q: lane j holds t_j, t_{j+32}, ...; row i of G is
// fetched one decision ahead.  Only what the next decision depends on sits in the loop (broadcast
// t_i, decide, one multiply-add per held entry); signs, norms and the non-finite check follow from
// the final t_j of every lane afterwards, in parallel.  Warp 0 only; rn2 = ||r||^2 before the
// step on entry, after it on return.
template <int Q>
__device__ __forceinline__ void scan_chain_regs(const ScanSmem &S, const double *G, int m, const CdgRule &rule,
                                                double &rn2, bool &bad, int &oob, int lane) {
  bool h[Q];
  double t[Q], g[Q], dg[Q];
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int j = lane + 32 * q;
    h[q] = j < m;
    t[q] = h[q] ? S.t[j] : 0.0;
    g[q] = h[q] ? G[j] : 0.0;
    dg[q] = h[q] ? G[(size_t)j * m + j] : 0.0;
  }
#pragma unroll
  for (int seg = 0; seg < Q; ++seg) {
    const int i_hi = (m < 32 * (seg + 1)) ? m : 32 * (seg + 1);
    for (int i = 32 * seg; i < i_hi; ++i) {
      double nx[Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) nx[q] = (i + 1 < m && h[q]) ? G[(size_t)(i + 1) * m + lane + 32 * q] : 0.0;
      const double ti = __shfl_sync(0xffffffffu, t[seg], i & 31);
      // Algorithm 6: +1 iff ||r + c|| < ||r - c||  <=>  <r,c> < 0 (or the randomized rule)
      int dummy = 0;
      const double sd = rule.randomized ? (double)cdg_decide(rule, i, ti, dummy) : ((ti < 0.0) ? 1.0 : -1.0);
      // every later t_j gains s_i G_ij, summed in the order i = 0, 1, ...
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        if (lane + 32 * q > i) t[q] = fma(sd, g[q], t[q]);
        g[q] = nx[q];
      }
    }
  }
  // lane j now holds t_j = <r_{j-1}, c_j> (and t_{j+32}, ...); its sign follows from it alone.
  // ||r||^2 seen by worker j: ||r_0||^2 + sum_{i<j} (2 s_i t_i + G_ii), an exclusive prefix sum over
  // the lanes, 32 workers after 32 workers
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int j = lane + 32 * q;
    const int sj = h[q] ? cdg_decide(rule, j, t[q], oob) : 0;
    bad = bad || (h[q] && !(isfinite(t[q]) && isfinite(dg[q])));
    const double inc = h[q] ? 2.0 * (double)sj * t[q] + dg[q] : 0.0;
    double pre = inc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, pre, off);
      if (lane >= off) pre += up;
    }
    const double before = rn2 + (pre - inc);
    if (h[q]) { S.s[j] = sj; S.rn[j] = before > 0.0 ? before : 0.0; S.t[j] = t[q]; }
    rn2 += __shfl_sync(0xffffffffu, pre, 31);
  }
  if (rn2 < 0.0) rn2 = 0.0;
  bad = __any_sync(0xffffffffu, bad);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) oob += __shfl_xor_sync(0xffffffffu, oob, off);
}

// S.t = b, S.p = pairs and G (shared or global, row-major [m][m]) must be ready and visible
// to the block (barrier before the call).  Warp 0 decides, the block writes out.
// rn2_in: ||r||^2 before the step when the caller fetched it ahead of time, else negative
// (the routine then reads *rnorm2 itself).  write_out = false: decide only (signs in S.s),
// nothing is written to global memory.  QMAX: lanes hold up to QMAX entries of the chain in
// registers (m <= 32 QMAX); beyond that the chain runs through shared memory.
template <int QMAX = 2>
__device__ __forceinline__ void scan_decide_and_write(const ScanSmem &S, const double *G, int m, int n, int k,
                                                      int32_t *__restrict__ perm_next, int8_t *__restrict__ signs,
                                                      float *__restrict__ margins, double *__restrict__ rnorm2,
                                                      int *__restrict__ status, const CdgRule rule,
                                                      double rn2_in = -1.0, bool write_out = true) {
  const int tid = threadIdx.x;
  if (tid < 32) {
    const int lane = tid;
    double rn2 = (rn2_in >= 0.0) ? rn2_in : *rnorm2;
    bool bad = false;
    int oob = 0;
    bool in_regs = false;
    if (m <= 64) {
      scan_chain_regs<2>(S, G, m, rule, rn2, bad, oob, lane);
      in_regs = true;
    }
    if constexpr (QMAX >= 4) {
      if (!in_regs && m <= 128) {
        scan_chain_regs<4>(S, G, m, rule, rn2, bad, oob, lane);
        in_regs = true;
      }
    }
    if (!in_regs) {
      for (int i = 0; i < m; ++i) {
        const double ti = S.t[i];
        const double gii = G[(size_t)i * m + i];
        const int s = cdg_decide(rule, i, ti, oob);
        bad |= !(isfinite(ti) && isfinite(gii));
        const double sd = (double)s;
        for (int j = i + 1 + lane; j < m; j += 32) S.t[j] += sd * G[(size_t)i * m + j];
        if (lane == 0) { S.s[i] = s; S.rn[i] = rn2; }
        rn2 += 2.0 * sd * ti + gii;
        if (rn2 < 0.0) rn2 = 0.0;
        __syncwarp();
      }
    }
    if (lane == 0 && write_out) {
      *rnorm2 = rn2;
      if (bad) atomicOr(status, CDG_ST_NONFINITE);
      if (oob) atomicAdd(rule.oob, (unsigned long long)oob);
    }
  }
  __syncthreads();
  if (!write_out) return;       // a replica of the decisions: S.s is all the caller needs
  const int half = n >> 1;
  for (int i = tid; i < m; i += blockDim.x) {
    if (!CDG_IDX_OK(k >= 0 && k < half, status)) continue;     // slots k and n-1-k of a row of n
    const int s = S.s[i];
    const size_t pos = (size_t)i * half + k;
    signs[pos] = (int8_t)s;
    const double den = S.rn[i] * G[(size_t)i * m + i];
    margins[pos] = (den > 0.0) ? (float)(fabs(S.t[i]) / sqrt(den)) : 0.f;
    // Algorithm 7: the item that received +1 goes to the front slot, the other to the back
    const int32_t first = S.p[2 * i], second = S.p[2 * i + 1];
    perm_next[(size_t)i * n + k] = (s == 1) ? first : second;
    perm_next[(size_t)i * n + (n - 1 - k)] = (s == 1) ? second : first;
  }
}
