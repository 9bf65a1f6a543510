// Internal declarations shared by the translation units of libcdgrab.so.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cdgrab.h"

#define CDG_MAGIC 0xCD62AB01u

// bits of the device status word
#define CDG_ST_NONFINITE 1
#define CDG_ST_TIMEOUT 2
#define CDG_ST_BOUNDS 4       // debug build: an index check failed (the write was skipped)

// Debug build (-DCDGRAB_DEBUG, python -m paper_2302_00845_b200.build --debug): index checks in
// front of the writes of the decision routines, and every handle-owned allocation wrapped in two
// guard blocks whose pattern cdgrab_status and cdgrab_destroy verify.  A failed check raises
// CDG_ST_BOUNDS and skips the write; nothing traps.
#ifdef CDGRAB_DEBUG
#define CDG_IDX_OK(cond, status) ((cond) ? true : (atomicOr((status), CDG_ST_BOUNDS), false))
#else
#define CDG_IDX_OK(cond, status) true
#endif
constexpr size_t kCdgGuardBytes = 256;
constexpr int kCdgMaxGuards = 32;
constexpr int kCdgGuardPattern = 0xA5;
struct CdgGuardRec { unsigned char *base; size_t bytes; };   // base: start of the head guard

// register tile edge of the generic FMA Gram kernel
#define CDG_TM 8
#define CDG_TILE_ENTRIES (CDG_TM * CDG_TM + CDG_TM)

// Tensor maps are encoded for a base address.  Callers alternate between a few gradient buffers
// (double buffering), so the maps of the last kCdgMapSlots bases are kept; a new base replaces
// the oldest entry.
constexpr int kCdgMapSlots = 4;
template <int N>
struct CdgMapCache {
  const void *base[kCdgMapSlots];
  CUtensorMap maps[kCdgMapSlots][N];
  int next;
  // slot holding the maps of `b`, or -1
  int find(const void *b) const {
    for (int i = 0; i < kCdgMapSlots; ++i)
      if (base[i] == b) return i;
    return -1;
  }
  // slot to encode the maps of a new base into (its old entry is forgotten until commit())
  int victim() { const int i = next; base[i] = nullptr; return i; }
  void commit(int i, const void *b) { base[i] = b; next = (i + 1) % kCdgMapSlots; }
};

struct cdgrab_ctx {
  uint32_t magic;
  int nguards;                          // debug build: guarded allocations of this handle
  CdgGuardRec guards[kCdgMaxGuards];
  int m, n;
  long long d;
  int dtype;
  int device;
  int num_sms;
  int path;          // CDGRAB_PATH_*
  int k;             // pairs consumed in the open epoch
  int epoch_open;
  long long launches;

  float *r;              // [d] running sum
  int32_t *perm_cur;     // [m][n]
  int32_t *perm_next;    // [m][n]
  int8_t *signs;         // [m][n/2]
  float *margins;        // [m][n/2]
  double *rnorm2;        // [1] tracked ||r||^2
  int *status;           // [1] device status word
  double *gram;          // [m*m + m] G (row-major) then b
  double *partials;      // pass-1 partial sums
  int shard;             // 1: this handle holds one column shard (split steps)
  int shard_pending;     // step_begin issued, step_finish outstanding
  int independent;       // 1: ID-GraB mode, r is [m][d] (one running sum per worker)
  int rule_randomized;   // balance rule of the step being enqueued (0: greedy)
  const float *rule_u;   // [m] uniforms for the randomized rule (NULL: seeded draws)
  unsigned long long rule_seed;
  unsigned rule_epoch;
  double rule_w;
  unsigned long long *oob;  // [1] positions with |<r,c>| > w seen by the randomized rule this epoch
  float *mean_out;       // [2][d] destination of the averaged gather buffers for the step being enqueued, or NULL
  size_t partials_bytes;
  int gram_chunks;       // grid.x of the FMA Gram kernels
  int gram_block;        // 1: the generic pass 1 is the blocked kernel (m > 16)

  // TMA-pipelined FMA Gram
  int fma_tma;             // 1 when that kernel serves pass 1
  int fma_tma_stages;
  int fma_tma_boxrows;     // rows per bulk-tensor copy
  int fma_tma_contig;      // 1: each CTA owns a contiguous range of tiles
  int upd_evict_first;     // pass 2 reads the rows with the L2 evict-first priority (256-bit loads)
  int pdl;                 // 1: dependent launches start early and wait on the device for their predecessor
  int cluster_off;         // 1: the one-launch step never spreads over a thread-block cluster (CDGRAB_CLUSTER=0)
  int fma_tma_fused;       // 1: the last CTA of pass 1 also combines and decides (no scan launch)
  unsigned *ticket;        // [1] arrival counter of the tensor-core path's hand-over, zero between launches
  int fma_tma_whole;       // 1: that launch also runs pass 2 (cooperative launch, no update launch)
  int ft_whole_launched;   // the last pass-1 launch was a whole step
  int ft_coop;             // 1: the whole-step launch is a cooperative launch
  int ft_coop_no_pdl;      // the driver refused cooperative + programmatic serialization together
  int ft_gsize;            // CTAs per group of the reduction tree
  unsigned long long ft_gen;          // launches of the tree so far (its counters only grow)
  unsigned long long *ft_ctr;         // [groups + 1] arrival counters of the tree
  double *ft_group_partials;          // [groups][152]
  size_t fma_tma_smem;
  int fma_tma_defer;       // 1: cdgrab_step_many folds pass 2 of a step into pass 1 of the next one
  int fma_tma_stages2;     // ring depth and shared memory of that form (a stage holds two steps' rows)
  size_t fma_tma_smem2;
  CUtensorMap tm_fr;       // 2-D map over r (one row)
  CdgMapCache<1> tm_fg;    // 2-D maps over the gradient rows of the last few buffers

  // optional per-kernel timing (cdgrab_profile_*): event pairs recorded around launches
  int prof_on;
  int prof_n, prof_cap;
  cudaEvent_t *prof_ev;    // [2 * prof_cap]
  int *prof_kind;          // [prof_cap]

  // tcgen05 path
  __nv_bfloat16 *r_split;  // [3][d_pad] hi/mid/lo parts of r
  long long d_pad;
  float *umma_partials;    // [ctas][128][ncols]
  int umma_ctas;
  int umma_box_rows;       // rows of the gradient TMA box (2m rounded up to 16)
  int umma_ncols;          // columns of a partial H row = box_rows + 16
  int umma_subs_per_stage;
  int umma_drain;          // pipeline iterations per TMEM accumulation chunk
  int umma_stages;
  size_t umma_smem;
  CUtensorMap tm_r;        // 3-D tensor map over r_split
  CUtensorMap tm_r2;       // 2-D map over r_split (ragged last block)
  CUtensorMap tm_r32;      // 2-D map over r itself (fp32), when pass 1 forms the bf16 rows in shared memory
  int umma_rconv;          // 1: pass 1 reads r as fp32 and splits it in the kernel (no r_split in HBM)
  int umma_rbox;           // 64-column blocks of r per fp32 copy
  // maps over the gradient rows of the last few buffers: [0] 3-D, [1] 2-D (ragged last block),
  // [2] 4-D over the full 8-row groups
  CdgMapCache<3> tm_g;
  int umma_g4;             // row groups one 4-D copy brings in (0: per-group copies only)
  int umma_paired;         // 2m <= 64: one MMA covers two 64-column blocks
  int umma_fused;          // the combine launch also takes the decisions (last block)
  int umma_rows;           // rows of the MMA operand: 2m

  // tcgen05 path for fp32 gradients with the bf16 terms formed inside the kernel
  int umma_f32;            // 1: that kernel serves pass 1
  int f32_nt;              // bf16 terms per difference: 3 (fp32 gradients) or 2 (bf16 gradients, m > 64)
  int f32_npad;            // MMA N: terms x m rounded up to 16
  int f32_nsub;            // 64-column blocks per stage
  int f32_nops;            // operand buffers
  int f32_stages;
  int f32_drain;           // 64-column blocks per TMEM accumulation chunk
  int f32_mma_m;           // MMA M of the term-splitting kernel: 64 for fp32 with m <= 32, else 128
  int f32_conv8;           // 1: eight converter warps where six would take 6 rows per thread and pass
  int f32_ctas;
  size_t f32_smem;
  double *f32_bpart;       // [ctas][128] per-CTA partial b
  double *f32_dsum;        // [128][256] the partial D summed over the CTAs
  CUtensorMap tm_f32r;     // 2-D map over r (one row)
  CdgMapCache<1> tm_f32g;  // 2-D maps over the gradient rows of the last few buffers
};

// Handle-owned device memory.  Release build: cudaMalloc / cudaFree.  Debug build: 256 guard bytes
// in front and behind, recorded in the handle.
template <typename P>
inline cudaError_t cdg_alloc(cdgrab_ctx *h, P **out, size_t bytes) {
#ifdef CDGRAB_DEBUG
  *out = nullptr;
  if (h->nguards >= kCdgMaxGuards) return cudaErrorMemoryAllocation;
  unsigned char *base = nullptr;
  cudaError_t e = cudaMalloc(&base, bytes + 2 * kCdgGuardBytes);
  if (e != cudaSuccess) return e;
  e = cudaMemset(base, kCdgGuardPattern, kCdgGuardBytes);
  if (e == cudaSuccess) e = cudaMemset(base + kCdgGuardBytes + bytes, kCdgGuardPattern, kCdgGuardBytes);
  if (e != cudaSuccess) { cudaFree(base); return e; }
  h->guards[h->nguards].base = base;
  h->guards[h->nguards].bytes = bytes;
  h->nguards++;
  *out = reinterpret_cast<P *>(base + kCdgGuardBytes);
  return cudaSuccess;
#else
  (void)h;
  return cudaMalloc(out, bytes);
#endif
}
inline void cdg_free(void *p) {
#ifdef CDGRAB_DEBUG
  if (p) cudaFree(static_cast<unsigned char *>(p) - kCdgGuardBytes);
#else
  cudaFree(p);
#endif
}
// index of the first allocation whose guard blocks no longer hold the pattern, -1 if all intact
// (always -1 in the release build); synchronous
int cdg_first_broken_guard(const cdgrab_ctx *h);

template <typename T>
__device__ __forceinline__ float cdg_ld(const T *p);
template <>
__device__ __forceinline__ float cdg_ld<float>(const float *p) { return *p; }
template <>
__device__ __forceinline__ float cdg_ld<__nv_bfloat16>(const __nv_bfloat16 *p) {
  return __bfloat162float(*p);
}

// The limit is per kernel, not per handle: handles of different shapes share a kernel, so the
// TMA-fed kernels are always opened up to the architecture's maximum (227 KB per CTA).
constexpr int kCdgMaxDynSmem = 227 * 1024;
template <typename K>
inline cudaError_t cdg_open_smem_limit(K *kernel) {
  cudaFuncAttributes fa;
  const cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kCdgMaxDynSmem - (int)fa.sharedSizeBytes);   // static and dynamic share the 227 KB
}

// cudaFuncSetAttribute acts on the device that is current at the call, so a raised dynamic
// shared-memory limit has to be set once per (kernel, device): one flag array per call site.
struct CdgPerDevice { unsigned char done[64]; };
template <typename K>
inline cudaError_t cdg_raise_smem_limit(CdgPerDevice &flags, int device, K *kernel, size_t bytes) {
  const bool tracked = device >= 0 && device < 64;
  if (tracked && flags.done[device]) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && tracked) flags.done[device] = 1;
  return e;
}

// Event pair around one launch when profiling is on; a full pool stops recording.
struct CdgProfScope {
  cdgrab_ctx *h; cudaStream_t st; int slot;
  CdgProfScope(cdgrab_ctx *h_, int kind, cudaStream_t st_) : h(h_), st(st_), slot(-1) {
    h->launches++;
    if (h->prof_on && h->prof_n < h->prof_cap) {
      slot = h->prof_n++;
      h->prof_kind[slot] = kind;
      cudaEventRecord(h->prof_ev[2 * slot], st);
    }
  }
  ~CdgProfScope() { if (slot >= 0) cudaEventRecord(h->prof_ev[2 * slot + 1], st); }
};

// Programmatic dependent launch.  A kernel launched through cdg_launch_dep may be scheduled while
// its predecessor in the stream is still running; it must call cdg_grid_dep_wait() before it
// touches anything the predecessor writes (the wait returns once that grid has completed and
// its writes are visible; without the launch attribute it returns at once).  A predecessor may
// call cdg_grid_dep_trigger() to let the successor's blocks take SMs as its own blocks leave.
#ifdef __CUDACC__
__device__ __forceinline__ void cdg_grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cdg_grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t cdg_launch_dep(const cdgrab_ctx *h, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                  cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = h->pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---- launchers (each returns a cudaError_t; every kernel launch sits in a CdgProfScope) ----------
cudaError_t cdg_launch_gram_generic(cdgrab_ctx *h, const void *grads, cudaStream_t st);
cudaError_t cdg_launch_gram_block(cdgrab_ctx *h, const void *grads, cudaStream_t st);   // m > 16: 64-row blocks
int cdg_block_ctas(const cdgrab_ctx *h);
size_t cdg_block_partials_bytes(const cdgrab_ctx *h);
cudaError_t cdg_launch_scan(cdgrab_ctx *h, cudaStream_t st);
cudaError_t cdg_launch_update(cdgrab_ctx *h, const void *grads, cudaStream_t st);
cudaError_t cdg_launch_mean(cdgrab_ctx *h, const void *grads, cudaStream_t st);
cudaError_t cdg_launch_split_r(cdgrab_ctx *h, cudaStream_t st);
cudaError_t cdg_launch_fused(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st);   // count steps, one launch
cudaError_t cdg_launch_gram_fma(cdgrab_ctx *h, const void *grads, cudaStream_t st);
cudaError_t cdg_launch_fused_logreg(cdgrab_ctx *h, const float *X, const float *y, const float *w, cudaStream_t st);
cudaError_t cdg_launch_logreg(cdgrab_ctx *h, const float *X, const float *y, const float *w,
                              float *out, cudaStream_t st);
bool cdg_fused_supported(int m, long long d, int dtype);
// the same single-launch Gram form for 17 <= m <= 128 workers whose step fits shared memory
bool cdg_small_supported(int m, long long d, int dtype);
cudaError_t cdg_launch_small(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st);
// the literal form: one CTA, Algorithm 6 worker by worker, count steps per launch (short rows, any m <= 1024)
bool cdg_literal_supported(int m, long long d, int dtype);
cudaError_t cdg_launch_literal(cdgrab_ctx *h, const void *grads, int count, cudaStream_t st);

// cuTensorMapEncodeTiled looked up through the runtime (NULL when the driver lacks it)
void *cdg_tensor_map_encoder();

// TMA-pipelined FMA Gram (m <= 16)
bool cdg_fma_tma_supported(int m, long long d, int dtype);
int cdg_fma_tma_setup(cdgrab_ctx *h);
cudaError_t cdg_launch_gram_fma_tma(cdgrab_ctx *h, const void *grads, cudaStream_t st);
// ... that first applies the open update of the step before (rows at grads_prev, signs at k - 1)
cudaError_t cdg_launch_gram_fma_tma_deferred(cdgrab_ctx *h, const void *grads, const void *grads_prev, cudaStream_t st);

// ID-GraB (independent workers)
int cdg_indep_chunks(const cdgrab_ctx *h);
cudaError_t cdg_launch_indep(cdgrab_ctx *h, const void *grads, cudaStream_t st);

cudaError_t cdg_launch_wait_selftest(cdgrab_ctx *h, long long cycles, long long *waited_dev, cudaStream_t st);

// tcgen05 path
bool cdg_umma_supported(int m, long long d, int dtype);
int cdg_umma_setup(cdgrab_ctx *h);   // allocations + tensor maps; CDGRAB_* code
void cdg_umma_teardown(cdgrab_ctx *h);
cudaError_t cdg_launch_gram_umma(cdgrab_ctx *h, const void *grads, cudaStream_t st);
// ... for fp32 gradients, terms formed in the kernel (17 <= m <= 64)
bool cdg_umma_f32_supported(int m, long long d);
bool cdg_umma_terms_bf16_supported(int m, long long d);   // the same kernel for bf16 gradients, 65 <= m <= 128
int cdg_umma_f32_setup(cdgrab_ctx *h);
void cdg_umma_f32_teardown(cdgrab_ctx *h);
cudaError_t cdg_launch_gram_umma_f32(cdgrab_ctx *h, const void *grads, cudaStream_t st);
