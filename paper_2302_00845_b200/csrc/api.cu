// C ABI of libcdgrab.so: handle life cycle, epoch state machine, path dispatch.
// Every step of the path runs in the kernels; this file only validates and enqueues.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"
#include "scan.cuh"

namespace {

inline bool valid(const cdgrab_ctx *h) { return h && h->magic == CDG_MAGIC; }

// A handle's buffers, tensor maps and kernel attributes belong to the device it was created on;
// work may only be enqueued while that device is current.
inline bool on_own_device(const cdgrab_ctx *h) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
  return dev == h->device;
}

inline size_t elem_size(int dtype) { return dtype == CDGRAB_F32 ? 4 : 2; }

__global__ void iota_perm_kernel(int32_t *p, int m, int n) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < (long long)m * n) p[idx] = (int32_t)(idx % n);
}

void free_all(cdgrab_ctx *h) {
  cdg_umma_teardown(h);
  cdg_free(h->r); cdg_free(h->perm_cur); cdg_free(h->perm_next); cdg_free(h->signs);
  cdg_free(h->margins); cdg_free(h->rnorm2); cdg_free(h->status); cdg_free(h->gram);
  cdg_free(h->partials);
  cdg_free(h->ticket);
  cdg_free(h->ft_ctr);
  cdg_free(h->ft_group_partials);
  cdg_free(h->oob);
  if (h->prof_ev) {
    for (int i = 0; i < 2 * h->prof_cap; ++i) if (h->prof_ev[i]) cudaEventDestroy(h->prof_ev[i]);
    free(h->prof_ev);
    free(h->prof_kind);
    h->prof_ev = nullptr; h->prof_kind = nullptr;
  }
}

int forced_path() {
  const char *e = getenv("CDGRAB_FORCE_PATH");
  if (!e || !*e || !strcmp(e, "auto")) return CDGRAB_PATH_AUTO;
  if (!strcmp(e, "fused")) return CDGRAB_PATH_FUSED;
  if (!strcmp(e, "fma")) return CDGRAB_PATH_FMA;
  if (!strcmp(e, "umma")) return CDGRAB_PATH_UMMA;
  if (!strcmp(e, "literal")) return CDGRAB_PATH_LITERAL;
  return -1;
}

inline bool fma_columns_ok(const cdgrab_ctx *h) { return h->m <= 16 && h->d % 4 == 0; }

int copy_out(void *dst, const void *src, size_t bytes, void *stream) {
  if (!dst) return CDGRAB_ERR_INVALID;
  if (cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  return CDGRAB_OK;
}

}  // namespace

int cdg_first_broken_guard(const cdgrab_ctx *h) {
#ifdef CDGRAB_DEBUG
  unsigned char buf[2 * kCdgGuardBytes];
  for (int g = 0; g < h->nguards; ++g) {
    const CdgGuardRec &rec = h->guards[g];
    if (cudaMemcpy(buf, rec.base, kCdgGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(buf + kCdgGuardBytes, rec.base + kCdgGuardBytes + rec.bytes, kCdgGuardBytes,
                   cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return g;
    }
    for (size_t i = 0; i < 2 * kCdgGuardBytes; ++i)
      if (buf[i] != kCdgGuardPattern) return g;
  }
#else
  (void)h;
#endif
  return -1;
}

#ifdef CDGRAB_DEBUG
// Debug build only: how many guarded allocations the handle has, and a HOST-side overwrite of one
// guard byte of allocation `which` (behind it when tail != 0), for the test of the guard check.
extern "C" int cdgrab_debug_guard_count(cdgrab_t *h) { return valid(h) ? h->nguards : CDGRAB_ERR_INVALID; }
extern "C" int cdgrab_debug_poke_guard(cdgrab_t *h, int which, int tail) {
  if (!valid(h) || which < 0 || which >= h->nguards) return CDGRAB_ERR_INVALID;
  const CdgGuardRec &rec = h->guards[which];
  unsigned char *p = tail ? rec.base + kCdgGuardBytes + rec.bytes : rec.base + kCdgGuardBytes - 1;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemset(p, 0, 1) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  return CDGRAB_OK;
}
#endif

extern "C" {

const char *cdgrab_strerror(int code) {
  switch (code) {
    case CDGRAB_OK: return "ok";
    case CDGRAB_ERR_INVALID: return "invalid argument";
    case CDGRAB_ERR_STATE: return "call not allowed in the current epoch state";
    case CDGRAB_ERR_CUDA: return "CUDA call failed";
    case CDGRAB_ERR_NOMEM: return "out of memory";
    case CDGRAB_ERR_NONFINITE: return "non-finite value met in a reduction";
    case CDGRAB_ERR_TIMEOUT: return "bounded device-side wait expired";
    case CDGRAB_ERR_DEVICE: return "no usable sm_100 CUDA device";
    case CDGRAB_ERR_TOO_LARGE: return "size beyond the fixed scratch of the no-allocation entry point";
    case CDGRAB_ERR_CORRUPT: return "guard bytes around library memory overwritten, or an index check failed (debug build)";
    default: return "unknown error";
  }
}

static int create_impl(int m, int n, long long d, int dtype, int mode, cdgrab_t **out);

int cdgrab_create(int m, int n, long long d, int dtype, cdgrab_t **out) {
  return create_impl(m, n, d, dtype, 0, out);
}

int cdgrab_create_independent(int m, int n, long long d, int dtype, cdgrab_t **out) {
  return create_impl(m, n, d, dtype, 1, out);
}

int cdgrab_create_shard(int m, int n, long long d_local, int dtype, cdgrab_t **out) {
  return create_impl(m, n, d_local, dtype, 2, out);
}

// mode 0: coordinated order on one device; 1: independent workers; 2: one column shard of a
// coordinated order (split steps, never the single-launch paths)
static int create_impl(int m, int n, long long d, int dtype, int mode, cdgrab_t **out) {
  const int independent = (mode == 1);
  const int shard = (mode == 2);
  if (!out) return CDGRAB_ERR_INVALID;
  *out = nullptr;
  if (m < 1 || m > 1024 || n < 2 || (n & 1) || d < 1) return CDGRAB_ERR_INVALID;
  if ((long long)m * n >= (1ll << 31)) return CDGRAB_ERR_INVALID;
  if (dtype != CDGRAB_F32 && dtype != CDGRAB_BF16) return CDGRAB_ERR_INVALID;
  const int forced = forced_path();
  if (forced < 0) return CDGRAB_ERR_INVALID;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_DEVICE; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_DEVICE; }
  if (prop.major != 10) return CDGRAB_ERR_DEVICE;  // the kernels are built for sm_100a only

  cdgrab_ctx *h = new (std::nothrow) cdgrab_ctx();
  if (!h) return CDGRAB_ERR_NOMEM;
  memset(h, 0, sizeof(*h));
  h->magic = CDG_MAGIC;
  h->m = m; h->n = n; h->d = d; h->dtype = dtype;
  h->device = dev; h->num_sms = prop.multiProcessorCount;
  h->independent = independent;
  h->shard = shard;
  h->pdl = 1;                      // CDGRAB_PDL=0: plain stream order between the launches of a step
  if (const char *e = getenv("CDGRAB_PDL")) h->pdl = atoi(e) ? 1 : 0;
  if (const char *e = getenv("CDGRAB_CLUSTER")) h->cluster_off = atoi(e) ? 0 : 1;
  // Pass 2 is the last reader of a step's rows.  Where a step is about the size of L2 (workload 3:
  // 128 MiB against 126 MB) reading them with the evict-first priority keeps them from pushing r
  // and the next step's first rows out: pass 2 took 24.8 instead of 30 us on a box where it paid
  // most; on steps many times L2 the hint cost 1-4 %, so it is tied to the step's size.
  // CDGRAB_UPD_EF=0/1 overrides.
  h->upd_evict_first = (2 * (size_t)m * (size_t)d * elem_size(dtype) <= ((size_t)192 << 20)) ? 1 : 0;
  if (const char *e = getenv("CDGRAB_UPD_EF")) h->upd_evict_first = atoi(e) ? 1 : 0;

  // ---- choose the path ------------------------------------------------------------
  const size_t step_bytes = 2 * (size_t)m * (size_t)d * elem_size(dtype);
  const bool fused_ok = cdg_fused_supported(m, d, dtype) || cdg_small_supported(m, d, dtype);
  // bf16 with 65..128 workers: the term-splitting tensor-core kernel (CDGRAB_UMMA_BF16_WIDE=0: not used)
  const char *wide_env = getenv("CDGRAB_UMMA_BF16_WIDE");
  const bool umma_wide = dtype == CDGRAB_BF16 && cdg_umma_terms_bf16_supported(m, d) && !(wide_env && atoi(wide_env) == 0);
  const bool umma_ok = cdg_umma_supported(m, d, dtype) || umma_wide;
  const bool literal_ok = cdg_literal_supported(m, d, dtype) && !shard && !independent;
  int path;
  if (forced == CDGRAB_PATH_AUTO) {
    // short rows: the literal form (one dot product per worker) beats the Gram form of the
    // single-launch step up to 1024 columns, and the four launches of the generic two-pass route
    // for more than 16 workers while m*d stays small (measured per step with cold caches: 10.2 against
    // 12.5 us at m = 4, d = 1024; 29.5 against 60.5 us at m = 32, d = 1024; 70 against 57 us at m = 64, d = 2048)
    // More than 16 workers with rows of at most 64 columns (the synthetic herding study: 16) take
    // the Gram form in one CTA instead: every dot product in parallel rather than one block-wide
    // reduction per worker (12.8 / 18.6 / 34.9 against 17.2 / 35.0 / 62.1 us per step at m = 20 /
    // 50 / 100, d = 16); with longer rows its one thread per entry loses to the literal form
    // (76 against 31 us at m = 32, d = 1024).
    const bool small_auto = cdg_small_supported(m, d, dtype) && d <= 64 && !shard;
    if (literal_ok && !small_auto && ((m <= 16 && d <= 1024) || (m > 16 && d < 4096 && (long long)m * d <= 65536)))
      path = CDGRAB_PATH_LITERAL;
    else if (small_auto || (cdg_fused_supported(m, d, dtype) && step_bytes <= (size_t)768 * 1024 && !shard))
      path = CDGRAB_PATH_FUSED;
    else if (umma_ok && !fma_columns_ok(h)) path = CDGRAB_PATH_UMMA;
    else path = CDGRAB_PATH_FMA;
  } else {
    path = forced;
    if ((path == CDGRAB_PATH_FUSED && (!fused_ok || shard)) || (path == CDGRAB_PATH_UMMA && !umma_ok) ||
        (path == CDGRAB_PATH_LITERAL && !literal_ok)) {
      delete h;
      return CDGRAB_ERR_INVALID;
    }
  }
  if (independent) path = CDGRAB_PATH_INDEPENDENT;
  h->path = path;

  // ---- allocations ----------------------------------------------------------------
  const size_t np = (size_t)m * (size_t)(n / 2);
  bool ok = true;
  const size_t r_elems = (size_t)d * (independent ? (size_t)m : 1);
  ok = ok && cdg_alloc(h, &h->r, sizeof(float) * r_elems) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->perm_cur, sizeof(int32_t) * (size_t)m * n) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->perm_next, sizeof(int32_t) * (size_t)m * n) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->signs, np) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->margins, sizeof(float) * np) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->rnorm2, sizeof(double)) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->status, sizeof(int)) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->gram, sizeof(double) * ((size_t)m * m + m)) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->oob, sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaMemset(h->oob, 0, sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cdg_alloc(h, &h->ticket, sizeof(unsigned)) == cudaSuccess;
  ok = ok && cudaMemset(h->ticket, 0, sizeof(unsigned)) == cudaSuccess;
  if (ok && independent) {
    h->gram_chunks = cdg_indep_chunks(h);
    h->partials_bytes = sizeof(double) * 3 * (size_t)m * (size_t)h->gram_chunks;
    ok = ok && cdg_alloc(h, &h->partials, h->partials_bytes) == cudaSuccess;
  }
  if (ok && path == CDGRAB_PATH_FMA) {
    if (fma_columns_ok(h)) {
      // thread-per-column kernel: one partial vector (<= 152 doubles) per block
      long long blocks = (d / 4 + 255) / 256;
      if (blocks > (long long)h->num_sms * 2) blocks = (long long)h->num_sms * 2;
      h->gram_chunks = (int)blocks;
      // sized for the larger of the two grids that may write it: this kernel's (<= 2 per SM)
      // and the TMA-fed kernel's (one CTA per SM whatever the row length)
      h->partials_bytes = sizeof(double) * 152 * (size_t)h->num_sms * 2;
    } else if (m > 16 && !(getenv("CDGRAB_GRAM_BLOCK") && atoi(getenv("CDGRAB_GRAM_BLOCK")) == 0)) {
      h->gram_block = 1;
      h->gram_chunks = cdg_block_ctas(h);
      h->partials_bytes = cdg_block_partials_bytes(h);
    } else {
      const int ntile = (m + CDG_TM - 1) / CDG_TM;
      const int npairs = ntile * (ntile + 1) / 2;
      long long chunks = (d + 256ll * 512 - 1) / (256ll * 512);  // <= 512 columns per thread
      const long long fill = (2ll * h->num_sms + npairs - 1) / npairs;
      const long long maxc = (d + 255) / 256;
      if (chunks < fill) chunks = fill;
      if (chunks > maxc) chunks = maxc;
      h->gram_chunks = (int)chunks;
      h->partials_bytes = sizeof(double) * CDG_TILE_ENTRIES * (size_t)npairs * (size_t)chunks;
    }
    ok = ok && cdg_alloc(h, &h->partials, h->partials_bytes) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    free_all(h);
    delete h;
    return CDGRAB_ERR_NOMEM;
  }
  if (path == CDGRAB_PATH_UMMA) {
    const int rc = umma_wide ? cdg_umma_f32_setup(h) : cdg_umma_setup(h);
    if (rc != CDGRAB_OK) { free_all(h); delete h; return rc; }
  }
  if (path == CDGRAB_PATH_FMA && fma_columns_ok(h) && cdg_fma_tma_supported(m, d, dtype)) {
    // CDGRAB_FMA_TMA=0 keeps the load-from-registers Gram kernel (diagnostic knob)
    const char *e = getenv("CDGRAB_FMA_TMA");
    if (!(e && e[0] == '0')) {
      const int rc = cdg_fma_tma_setup(h);
      if (rc != CDGRAB_OK) { free_all(h); delete h; return rc; }
      if (shard) h->fma_tma_fused = 0;   // the decisions wait for the sum over all shards
    }
  }

  const long long tot = (long long)m * n;
  iota_perm_kernel<<<(unsigned)((tot + 255) / 256), 256>>>(h->perm_cur, m, n);
  cudaMemset(h->perm_next, 0, sizeof(int32_t) * (size_t)m * n);
  cudaMemset(h->signs, 0, np);
  cudaMemset(h->margins, 0, sizeof(float) * np);
  cudaMemset(h->rnorm2, 0, sizeof(double));
  cudaMemset(h->status, 0, sizeof(int));
  cudaMemset(h->r, 0, sizeof(float) * r_elems);
  if (cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    free_all(h);
    delete h;
    return CDGRAB_ERR_CUDA;
  }
  *out = h;
  return CDGRAB_OK;
}

int cdgrab_destroy(cdgrab_t *h) {
  if (!h) return CDGRAB_OK;
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  cudaDeviceSynchronize();
  const int rc = cdg_first_broken_guard(h) >= 0 ? CDGRAB_ERR_CORRUPT : CDGRAB_OK;   // debug build only
  free_all(h);
  h->magic = 0;
  delete h;
  return rc;
}

int cdgrab_set_perms(cdgrab_t *h, const int32_t *perms_in) {
  if (!valid(h) || !perms_in) return CDGRAB_ERR_INVALID;
  if (h->epoch_open) return CDGRAB_ERR_STATE;
  const size_t cnt = (size_t)h->m * h->n;
  std::vector<int32_t> host(cnt);
  if (cudaMemcpy(host.data(), perms_in, cnt * sizeof(int32_t), cudaMemcpyDefault) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  std::vector<char> seen(h->n);
  for (int i = 0; i < h->m; ++i) {
    std::fill(seen.begin(), seen.end(), 0);
    for (int j = 0; j < h->n; ++j) {
      const int32_t v = host[(size_t)i * h->n + j];
      if (v < 0 || v >= h->n || seen[v]) return CDGRAB_ERR_INVALID;
      seen[v] = 1;
    }
  }
  if (cudaMemcpy(h->perm_cur, host.data(), cnt * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  return CDGRAB_OK;
}

int cdgrab_begin_epoch(cdgrab_t *h, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (h->epoch_open) return CDGRAB_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(h->r, 0, sizeof(float) * (size_t)h->d * (h->independent ? (size_t)h->m : 1), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->rnorm2, 0, sizeof(double), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->oob, 0, sizeof(unsigned long long), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->signs, 0, (size_t)h->m * (h->n / 2), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->margins, 0, sizeof(float) * (size_t)h->m * (h->n / 2), st);
  if (e == cudaSuccess && h->r_split)
    e = cudaMemsetAsync(h->r_split, 0, sizeof(__nv_bfloat16) * 3 * (size_t)h->d_pad, st);
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->k = 0;
  h->epoch_open = 1;
  return CDGRAB_OK;
}

static cudaError_t launch_pass1(cdgrab_ctx *h, const void *grads_dev, cudaStream_t st) {
  if (h->path == CDGRAB_PATH_UMMA && h->umma_f32) return cdg_launch_gram_umma_f32(h, grads_dev, st);
  if (h->path == CDGRAB_PATH_UMMA) return cdg_launch_gram_umma(h, grads_dev, st);
  if (h->fma_tma) return cdg_launch_gram_fma_tma(h, grads_dev, st);
  if (fma_columns_ok(h)) return cdg_launch_gram_fma(h, grads_dev, st);
  return cdg_launch_gram_generic(h, grads_dev, st);
}

int cdgrab_step_begin(cdgrab_t *h, const void *grads_dev, double *gram_out_dev, void *stream) {
  if (!valid(h) || !grads_dev || !gram_out_dev || !h->shard) return CDGRAB_ERR_INVALID;
  if ((((uintptr_t)grads_dev & 15) | ((uintptr_t)gram_out_dev & 7)) != 0) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || h->k >= h->n / 2 || h->shard_pending) return CDGRAB_ERR_STATE;
  double *own = h->gram;
  h->gram = gram_out_dev;                       // pass 1 leaves this shard's partial (G, b) there
  const cudaError_t e = launch_pass1(h, grads_dev, (cudaStream_t)stream);
  h->gram = own;
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->shard_pending = 1;
  return CDGRAB_OK;
}

int cdgrab_step_finish(cdgrab_t *h, const void *grads_dev, const double *gram_in_dev, void *stream) {
  if (!valid(h) || !grads_dev || !gram_in_dev || !h->shard) return CDGRAB_ERR_INVALID;
  // pass 2 reads the rows with 16-byte vector loads, the scan reads doubles
  if ((((uintptr_t)grads_dev & 15) | ((uintptr_t)gram_in_dev & 7)) != 0) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || !h->shard_pending) return CDGRAB_ERR_STATE;
  double *own = h->gram;
  h->gram = const_cast<double *>(gram_in_dev);  // the sum over all shards
  cudaError_t e = cdg_launch_scan(h, (cudaStream_t)stream);
  h->gram = own;
  if (e == cudaSuccess) e = cdg_launch_update(h, grads_dev, (cudaStream_t)stream);
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->shard_pending = 0;
  h->k++;
  return CDGRAB_OK;
}

int cdgrab_step(cdgrab_t *h, const void *grads_dev, void *stream) {
  if (!valid(h) || !grads_dev) return CDGRAB_ERR_INVALID;
  if (((uintptr_t)grads_dev & 15) != 0) return CDGRAB_ERR_INVALID;
  if (h->shard) return CDGRAB_ERR_INVALID;   // a shard steps through cdgrab_step_begin / _finish
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || h->k >= h->n / 2) return CDGRAB_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (h->independent) {
    if (h->rule_randomized || h->mean_out) return CDGRAB_ERR_INVALID;  // greedy rule only in this mode
    e = cdg_launch_indep(h, grads_dev, st);
  } else if (h->path == CDGRAB_PATH_FUSED) {
    e = h->m > 16 ? cdg_launch_small(h, grads_dev, 1, st) : cdg_launch_fused(h, grads_dev, 1, st);
  } else if (h->path == CDGRAB_PATH_LITERAL) {
    e = cdg_launch_literal(h, grads_dev, 1, st);
  } else {
    e = launch_pass1(h, grads_dev, st);
    const bool decided = (h->path == CDGRAB_PATH_UMMA) ? h->umma_fused : (h->fma_tma && h->fma_tma_fused);
    if (e == cudaSuccess && !decided) e = cdg_launch_scan(h, st);
    const bool updated = h->fma_tma && h->ft_whole_launched;     // pass 2 ran inside the pass-1 launch
    if (e == cudaSuccess && !updated) e = cdg_launch_update(h, grads_dev, st);
  }
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->k++;
  return CDGRAB_OK;
}

int cdgrab_step_many(cdgrab_t *h, const void *grads_dev, int count, void *stream) {
  if (!valid(h) || !grads_dev || count < 1) return CDGRAB_ERR_INVALID;
  if (((uintptr_t)grads_dev & 15) != 0 || h->shard) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || h->k + count > h->n / 2) return CDGRAB_ERR_STATE;
  const size_t step_bytes = 2 * (size_t)h->m * (size_t)h->d * (h->dtype == CDGRAB_F32 ? 4 : 2);
  if (h->path == CDGRAB_PATH_FUSED && !h->independent && !h->rule_randomized && !h->mean_out) {
    if (step_bytes % 16 != 0) return CDGRAB_ERR_INVALID;
    const cudaError_t e = h->m > 16 ? cdg_launch_small(h, grads_dev, count, (cudaStream_t)stream)
                                    : cdg_launch_fused(h, grads_dev, count, (cudaStream_t)stream);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return CDGRAB_ERR_CUDA;
    }
    h->k += count;
    return CDGRAB_OK;
  }
  // Deferred update (TMA-fed FMA path): pass 1 of step j also applies the update step j - 1 left
  // open, so the call takes count + 1 streaming launches instead of 2 count and reads r once per
  // step; only the last step's update gets a launch of its own.
  if (count > 1 && h->path == CDGRAB_PATH_FMA && h->fma_tma && h->fma_tma_fused && h->fma_tma_defer &&
      !h->independent && !h->rule_randomized && !h->mean_out) {
    cudaStream_t st = (cudaStream_t)stream;
    const char *g = (const char *)grads_dev;
    cudaError_t e = cdg_launch_gram_fma_tma(h, g, st);
    for (int i = 1; i < count && e == cudaSuccess; ++i) {
      h->k++;                               // the step whose decisions this launch takes
      e = cdg_launch_gram_fma_tma_deferred(h, g + (size_t)i * step_bytes, g + (size_t)(i - 1) * step_bytes, st);
    }
    if (e == cudaSuccess) e = cdg_launch_update(h, g + (size_t)(count - 1) * step_bytes, st);
    if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
    h->k++;
    return CDGRAB_OK;
  }
  if (h->path == CDGRAB_PATH_LITERAL && !h->rule_randomized && !h->mean_out) {
    if (step_bytes % 16 != 0) return CDGRAB_ERR_INVALID;
    if (cdg_launch_literal(h, grads_dev, count, (cudaStream_t)stream) != cudaSuccess) {
      cudaGetLastError();
      return CDGRAB_ERR_CUDA;
    }
    h->k += count;
    return CDGRAB_OK;
  }
  for (int i = 0; i < count; ++i) {
    const int rc = cdgrab_step(h, (const char *)grads_dev + (size_t)i * step_bytes, stream);
    if (rc != CDGRAB_OK) return rc;
  }
  return CDGRAB_OK;
}

int cdgrab_step_logreg(cdgrab_t *h, const float *X, const float *y, const float *w, void *stream) {
  if (!valid(h) || !X || !y || !w) return CDGRAB_ERR_INVALID;
  // the one-launch step from feature rows serves handles on either single-launch path
  const bool single = (h->path == CDGRAB_PATH_FUSED || h->path == CDGRAB_PATH_LITERAL) &&
                      cdg_fused_supported(h->m, h->d, h->dtype);
  if (h->dtype != CDGRAB_F32 || !single) return CDGRAB_ERR_INVALID;
  if ((((uintptr_t)X | (uintptr_t)w) & 15) != 0) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || h->k >= h->n / 2) return CDGRAB_ERR_STATE;
  if (cdg_launch_fused_logreg(h, X, y, w, (cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->k++;
  return CDGRAB_OK;
}

int cdgrab_step_randomized(cdgrab_t *h, const void *grads_dev, const float *u_dev, double w, void *stream) {
  if (!valid(h) || !u_dev || !(w > 0.0)) return CDGRAB_ERR_INVALID;
  h->rule_randomized = 1; h->rule_u = u_dev; h->rule_w = w;
  const int rc = cdgrab_step(h, grads_dev, stream);
  h->rule_randomized = 0; h->rule_u = nullptr; h->rule_w = 0.0;
  return rc;
}

int cdgrab_step_randomized_seeded(cdgrab_t *h, const void *grads_dev, unsigned long long seed, unsigned epoch,
                                  double w, void *stream) {
  if (!valid(h) || !(w > 0.0)) return CDGRAB_ERR_INVALID;
  h->rule_randomized = 1; h->rule_u = nullptr; h->rule_w = w; h->rule_seed = seed; h->rule_epoch = epoch;
  const int rc = cdgrab_step(h, grads_dev, stream);
  h->rule_randomized = 0; h->rule_w = 0.0;
  return rc;
}

namespace {
__global__ void seeded_uniforms_kernel(unsigned long long seed, unsigned epoch, unsigned k, int m, float *out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < m) out[i] = cdg_seeded_uniform(seed, epoch, k, (unsigned)i);
}
}  // namespace

int cdgrab_randomized_uniforms(unsigned long long seed, unsigned epoch, unsigned k, int m, float *u_out_dev,
                               void *stream) {
  if (m < 1 || !u_out_dev) return CDGRAB_ERR_INVALID;
  seeded_uniforms_kernel<<<(m + 127) / 128, 128, 0, (cudaStream_t)stream>>>(seed, epoch, k, m, u_out_dev);
  if (cudaGetLastError() != cudaSuccess) return CDGRAB_ERR_CUDA;
  return CDGRAB_OK;
}

long long cdgrab_out_of_bound(cdgrab_t *h) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  unsigned long long v = 0;
  if (cudaMemcpy(&v, h->oob, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  return (long long)v;
}

int cdgrab_step_mean(cdgrab_t *h, const void *grads_dev, float *mean_out_dev, void *stream) {
  if (!valid(h) || !mean_out_dev) return CDGRAB_ERR_INVALID;
  if (((uintptr_t)mean_out_dev & 15) != 0) return CDGRAB_ERR_INVALID;   // written with 16-byte vector stores
  h->mean_out = mean_out_dev;
  int rc = cdgrab_step(h, grads_dev, stream);
  if (rc == CDGRAB_OK && (h->path == CDGRAB_PATH_FUSED || h->path == CDGRAB_PATH_LITERAL)) {
    // the single-launch steps have no separate pass 2 to fold the average into
    if (cdg_launch_mean(h, grads_dev, (cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); rc = CDGRAB_ERR_CUDA; }
  }
  h->mean_out = nullptr;
  return rc;
}

int cdgrab_step_host(cdgrab_t *h, const void *grads_host, void *staging_dev, void *stream) {
  if (!valid(h) || !grads_host || !staging_dev) return CDGRAB_ERR_INVALID;
  if (((uintptr_t)staging_dev & 15) != 0) return CDGRAB_ERR_INVALID;
  if (!h->epoch_open || h->k >= h->n / 2) return CDGRAB_ERR_STATE;
  const size_t bytes = 2 * (size_t)h->m * (size_t)h->d * elem_size(h->dtype);
  if (cudaMemcpyAsync(staging_dev, grads_host, bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  return cdgrab_step(h, staging_dev, stream);
}

int cdgrab_end_epoch(cdgrab_t *h, int32_t *perms_out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (!h->epoch_open || h->k != h->n / 2 || h->shard_pending) return CDGRAB_ERR_STATE;
  int32_t *t = h->perm_cur; h->perm_cur = h->perm_next; h->perm_next = t;
  h->epoch_open = 0;
  if (perms_out) return copy_out(perms_out, h->perm_cur, sizeof(int32_t) * (size_t)h->m * h->n, stream);
  return CDGRAB_OK;
}

int cdgrab_get_signs(cdgrab_t *h, int8_t *out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->signs, (size_t)h->m * (h->n / 2), stream);
}
int cdgrab_get_r(cdgrab_t *h, float *out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->r, sizeof(float) * (size_t)h->d, stream);
}
int cdgrab_get_r_worker(cdgrab_t *h, int worker, float *out, void *stream) {
  if (!valid(h) || !h->independent || worker < 0 || worker >= h->m) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->r + (size_t)worker * (size_t)h->d, sizeof(float) * (size_t)h->d, stream);
}
int cdgrab_get_margins(cdgrab_t *h, float *out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->margins, sizeof(float) * (size_t)h->m * (h->n / 2), stream);
}
int cdgrab_get_perms(cdgrab_t *h, int32_t *out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->perm_cur, sizeof(int32_t) * (size_t)h->m * h->n, stream);
}
int cdgrab_get_next_perms(cdgrab_t *h, int32_t *out, void *stream) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  return copy_out(out, h->perm_next, sizeof(int32_t) * (size_t)h->m * h->n, stream);
}

int cdgrab_status(cdgrab_t *h) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  int st = 0;
  if (cudaMemcpy(&st, h->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  if (st & CDG_ST_BOUNDS) return CDGRAB_ERR_CORRUPT;
  if (cdg_first_broken_guard(h) >= 0) return CDGRAB_ERR_CORRUPT;
  if (st & CDG_ST_TIMEOUT) return CDGRAB_ERR_TIMEOUT;
  if (st & CDG_ST_NONFINITE) return CDGRAB_ERR_NONFINITE;
  return CDGRAB_OK;
}

int cdgrab_profile_enable(cdgrab_t *h, int on) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (on && !h->prof_ev) {
    const int cap = 8192;
    h->prof_ev = (cudaEvent_t *)calloc(2 * (size_t)cap, sizeof(cudaEvent_t));
    h->prof_kind = (int *)calloc(cap, sizeof(int));
    if (!h->prof_ev || !h->prof_kind) return CDGRAB_ERR_NOMEM;
    h->prof_cap = cap;
    for (int i = 0; i < 2 * cap; ++i)
      if (cudaEventCreate(&h->prof_ev[i]) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  }
  if (on) h->prof_n = 0;
  h->prof_on = on ? 1 : 0;
  return CDGRAB_OK;
}

int cdgrab_profile_read(cdgrab_t *h, int kind, double *total_ms, long long *launches) {
  if (!valid(h) || !total_ms || !launches || kind < 0 || kind >= CDGRAB_K_COUNT) return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  double tot = 0.0;
  long long cnt = 0;
  for (int i = 0; i < h->prof_n; ++i) {
    if (h->prof_kind[i] != kind) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]) != cudaSuccess) {
      cudaGetLastError();
      return CDGRAB_ERR_CUDA;
    }
    tot += ms;
    ++cnt;
  }
  *total_ms = tot;
  *launches = cnt;
  return CDGRAB_OK;
}

int cdgrab_selftest_wait_timeout(cdgrab_t *h, long long cycles, long long *waited_cycles) {
  if (!valid(h) || cycles < 1 || cycles > 2000000000ll) return CDGRAB_ERR_INVALID;
  long long *dev = nullptr;
  if (cudaMalloc(&dev, sizeof(long long)) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_NOMEM; }
  int rc = CDGRAB_OK;
  long long waited = 0;
  if (cdg_launch_wait_selftest(h, cycles, dev, nullptr) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&waited, dev, sizeof(long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    rc = CDGRAB_ERR_CUDA;
  }
  cudaFree(dev);
  if (waited_cycles) *waited_cycles = waited;
  return rc;
}

int cdgrab_clear_status(cdgrab_t *h) {
  if (!valid(h)) return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemset(h->status, 0, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  // a launch that gave up may have left the arrival counters of the reduction tree short
  if (h->ft_ctr) {
    if (cudaMemset(h->ft_ctr, 0, sizeof(unsigned long long) * 65) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
    h->ft_gen = 0;
  }
  if (h->ticket && cudaMemset(h->ticket, 0, sizeof(unsigned)) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  return CDGRAB_OK;
}

// ---- checkpoint / resume -----------------------------------------------------------------
namespace {
struct StateHeader {
  uint32_t magic;
  int m, n, dtype, independent, k, epoch_open;
  long long d;
  double rnorm2;
  unsigned long long oob;
};
struct StateSizes { size_t r, perm, signs, margins, total; };
StateSizes state_sizes(const cdgrab_ctx *h) {
  StateSizes z;
  z.r = sizeof(float) * (size_t)h->d * (h->independent ? (size_t)h->m : 1);
  z.perm = sizeof(int32_t) * (size_t)h->m * h->n;
  z.signs = (size_t)h->m * (h->n / 2);
  z.margins = sizeof(float) * (size_t)h->m * (h->n / 2);
  z.total = sizeof(StateHeader) + z.r + 2 * z.perm + z.signs + z.margins;
  return z;
}
}  // namespace

long long cdgrab_state_bytes(const cdgrab_t *h) { return valid(h) ? (long long)state_sizes(h).total : CDGRAB_ERR_INVALID; }

int cdgrab_save_state(cdgrab_t *h, void *host_buf, long long bytes) {
  if (!valid(h) || !host_buf) return CDGRAB_ERR_INVALID;
  const StateSizes z = state_sizes(h);
  if (bytes < (long long)z.total) return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  StateHeader hd;
  memset(&hd, 0, sizeof(hd));
  hd.magic = CDG_MAGIC; hd.m = h->m; hd.n = h->n; hd.dtype = h->dtype; hd.independent = h->independent;
  hd.k = h->k; hd.epoch_open = h->epoch_open; hd.d = h->d;
  char *p = (char *)host_buf + sizeof(StateHeader);
  bool ok = cudaMemcpy(&hd.rnorm2, h->rnorm2, sizeof(double), cudaMemcpyDeviceToHost) == cudaSuccess;
  ok = ok && cudaMemcpy(&hd.oob, h->oob, sizeof(hd.oob), cudaMemcpyDeviceToHost) == cudaSuccess;
  ok = ok && cudaMemcpy(p, h->r, z.r, cudaMemcpyDeviceToHost) == cudaSuccess; p += z.r;
  ok = ok && cudaMemcpy(p, h->perm_cur, z.perm, cudaMemcpyDeviceToHost) == cudaSuccess; p += z.perm;
  ok = ok && cudaMemcpy(p, h->perm_next, z.perm, cudaMemcpyDeviceToHost) == cudaSuccess; p += z.perm;
  ok = ok && cudaMemcpy(p, h->signs, z.signs, cudaMemcpyDeviceToHost) == cudaSuccess; p += z.signs;
  ok = ok && cudaMemcpy(p, h->margins, z.margins, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  memcpy(host_buf, &hd, sizeof(hd));
  return CDGRAB_OK;
}

int cdgrab_load_state(cdgrab_t *h, const void *host_buf, long long bytes) {
  if (!valid(h) || !host_buf) return CDGRAB_ERR_INVALID;
  const StateSizes z = state_sizes(h);
  if (bytes < (long long)z.total) return CDGRAB_ERR_INVALID;
  StateHeader hd;
  memcpy(&hd, host_buf, sizeof(hd));
  if (hd.magic != CDG_MAGIC || hd.m != h->m || hd.n != h->n || hd.d != h->d || hd.dtype != h->dtype ||
      hd.independent != h->independent || hd.k < 0 || hd.k > h->n / 2)
    return CDGRAB_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  const char *p = (const char *)host_buf + sizeof(StateHeader);
  bool ok = cudaMemcpy(h->rnorm2, &hd.rnorm2, sizeof(double), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(h->oob, &hd.oob, sizeof(hd.oob), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(h->r, p, z.r, cudaMemcpyHostToDevice) == cudaSuccess; p += z.r;
  ok = ok && cudaMemcpy(h->perm_cur, p, z.perm, cudaMemcpyHostToDevice) == cudaSuccess; p += z.perm;
  ok = ok && cudaMemcpy(h->perm_next, p, z.perm, cudaMemcpyHostToDevice) == cudaSuccess; p += z.perm;
  ok = ok && cudaMemcpy(h->signs, p, z.signs, cudaMemcpyHostToDevice) == cudaSuccess; p += z.signs;
  ok = ok && cudaMemcpy(h->margins, p, z.margins, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cdg_launch_split_r(h, nullptr) == cudaSuccess;
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  h->k = hd.k;
  h->epoch_open = hd.epoch_open;
  return CDGRAB_OK;
}

int cdgrab_path(const cdgrab_t *h) { return valid(h) ? h->path : CDGRAB_ERR_INVALID; }

long long cdgrab_launch_count(const cdgrab_t *h) { return valid(h) ? h->launches : -1; }

int cdgrab_logreg_grads(cdgrab_t *h, const float *X, const float *y, const float *w, float *grads_out,
                        void *stream) {
  if (!valid(h) || !X || !y || !w || !grads_out) return CDGRAB_ERR_INVALID;
  if (h->dtype != CDGRAB_F32) return CDGRAB_ERR_INVALID;
  if (!on_own_device(h)) return CDGRAB_ERR_DEVICE;
  if (!h->epoch_open || h->k >= h->n / 2) return CDGRAB_ERR_STATE;
  if (cdg_launch_logreg(h, X, y, w, grads_out, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  return CDGRAB_OK;
}

}  // extern "C"
