// Pass 1 on the tensor cores (tcgen05) with the pair differences split into bf16 terms inside the
// kernel: fp32 gradients with 17 <= m <= 64 (three terms), and bf16 gradients with 65 <= m <= 128
// (two terms; their 2m raw rows no longer fit one 128-row MMA tile).  The fp32 case first:
//
// The pair differences c_i = z1_i - z2_i (rounded to fp32, as every other path forms them) are
// written as three bf16 terms hi + mid + lo = c exactly (3 x 8 significand bits).  Products of
// bf16 terms are exact in the fp32 accumulator, so <c_k, c_i> is the sum of the nine term
// products; the lo x lo one (below 2^-32 of the product) is left out, the other eight come out
// of ONE product per 16 columns:  D = A B^T with B = [hi_0..hi_{m-1} | mid_0.. | lo_0..] (3m
// rows, the MMA's N) and A = the first 128 of those rows (hi and mid, the MMA's M; M = 64 when
// 2m <= 64, which halves the A bytes each MMA reads from shared memory):
//     G_ki = D[k][i] + D[k][m+i] + D[k][2m+i] + D[m+k][i] + D[m+k][m+i] + D[m+k][2m+i]
//            + D[i][2m+k] + D[m+i][2m+k]          (the last two are lo_k x hi_i and lo_k x mid_i).
// The terms are formed inside the kernel: TMA brings fp32 tiles [2m rows][64 s columns] and the
// matching piece of r into a ring of stages; six (or eight) converter warps read them, subtract, split,
// and store the bf16 terms into an operand buffer in the K-major 128-byte-swizzled layout the
// MMA reads ([8-row group][8 rows][128 B], 16-byte chunk c of row q at chunk c ^ (q & 7)).  The
// same warps add up b_i = <r, c_i> on the FMA pipe (fp32 products, moved into fp64 every 32
// blocks), so r needs no bf16 copy on this path.  Nothing but the caller's rows and r is read
// from HBM: 2mde + 4d bytes per launch.
//
// Roles (512 or 576 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2..7
// (2..9) converters, the last eight warps read the accumulator back.  The sum stays in TMEM for `drain` blocks
// of 64 columns only (the tensor core's fp32 accumulation truncates), then the read-back warps
// add the chunk to fp32 registers (round to nearest) while the MMAs fill the other buffer.
// One persistent CTA per SM owns a contiguous range of 64-column blocks; its partial D and b
// go to global memory, a second kernel adds the CTAs in index order in fp64, forms G and takes
// the step's decisions.  Every wait is bounded: on expiry the CTA raises the time-out bit of the
// status word, lets its copies land, frees its TMEM and returns.
//
// bf16 gradients, 65 <= m <= 128 (NT = 2): c = z1 - z2 in fp32, then c = hi + lo with a residual
// below 2^-17 |c| (the tolerance for bf16 inputs is 1e-3).  B = [hi_0.. | lo_0..] (N = 2m <= 256),
// A = the first 128 rows (all of hi), and  G_ki = D[k][i] + D[k][m+i] + D[i][m+k]  (hi x hi,
// hi x lo and its transpose; lo x lo, below 2^-16 of the product, is left out).  The converter
// threads take the rows in two passes to bound their registers, and the read-back warps add
// each chunk (4096 columns) to the CTA's partial D in global memory (it stays in L2) instead of
// holding 256 columns of accumulators in registers.
#include <cudaTypedefs.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"
#include "scan.cuh"

namespace {

// Converter warps: CW = 6 (12 rows of a 64-column block at a time) or CW = 8 (16 rows at a time).
// Eight pay where six would leave a thread six rows per pass (fp32 with more than 60 workers, bf16
// with more than 112): pass 1 measured 8 % (fp32, m = 64) and 13 % (bf16, m = 128) faster.  Where
// six warps take five rows each the two forms tie or eight lose a few per cent (m = 56, 100, 112),
// below that eight lose outright (idle row slots, warps waiting on one another).
constexpr int kDrainWarps = 8;
__host__ __device__ constexpr int terms_threads(int cw) { return 64 + 32 * cw + 32 * kDrainWarps; }
__host__ __device__ constexpr int terms_conv_rows(int cw) { return 2 * cw; }          // 16 threads (float4 each) per row of a block
constexpr int kMaxStages = 8;
constexpr int kMaxOps = 4;                           // operand buffers (one 64-column block each)
constexpr int kBlockCols = 64;                       // columns per MMA block = one 128-byte swizzle row of bf16
constexpr int kFlushBlocks = 32;                     // blocks between two moves of the fp32 b sums into fp64
constexpr int kMaxN = 256;                           // row pitch of the summed D: 3 m at m = 64, 2 m at m = 128
constexpr int kMaxM = 128;

struct F32Params {
  int m;
  int npad;            // MMA N: 3m rounded up to 16
  int nsub;            // 64-column blocks per stage
  int stages;
  int nops;            // operand buffers
  int drain;           // blocks accumulated in TMEM before the sum is read back
  long long nblk;      // ceil(d / 64)
  int pass_rows;       // rows per converter pass (a multiple of 8; = m rounded up when there is one pass)
  int mma_m;           // MMA M: 128, or 64 when the 2m rows of A fit (half the A bytes read from shared memory per MMA)
};

template <typename T>
struct TermIn;
template <>
struct TermIn<float> {                     // 4 columns = 16 bytes
  static __device__ __forceinline__ void ld(const uint8_t *p, float (&v)[4]) {
    const float4 f = *reinterpret_cast<const float4 *>(p);
    v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
  }
};
template <>
struct TermIn<__nv_bfloat16> {             // 4 columns = 8 bytes, widened exactly
  static __device__ __forceinline__ void ld(const uint8_t *p, float (&v)[4]) {
    const uint2 w = *reinterpret_cast<const uint2 *>(p);
    v[0] = __uint_as_float(w.x << 16); v[1] = __uint_as_float(w.x & 0xffff0000u);
    v[2] = __uint_as_float(w.y << 16); v[3] = __uint_as_float(w.y & 0xffff0000u);
  }
};

__device__ __forceinline__ uint64_t f32_umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for this layout)
  d |= (uint64_t)(1024u >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}
__device__ __forceinline__ void f32_umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ bool f32_elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void f32_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Bounded wait like mbar_wait, with a suspend-time hint: a waiting warp (producer, MMA issuer,
// read-back) sleeps in the barrier unit for up to a microsecond at a time instead of polling, and
// leaves the issue slots of its scheduler to the converter warps (-2 % on pass 1 at m = 32).
__device__ __forceinline__ bool f32_wait(uint32_t bar, uint32_t parity, long long deadline) {
  while (true) {
    uint32_t done;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(done) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    if (done) return true;
    if (clock64() > deadline) return false;
  }
}

// two floats rounded to bf16 (to nearest even), x in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float x, float y) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<const uint32_t *>(&h);
}

// T: element type of the gradients; NT: bf16 terms per difference; NP: passes the converter
// threads make over the rows of a block; NS: rows each converter thread takes per pass, a
// compile-time count so that the NS x 2 split chains sit in one basic block and the scheduler
// can interleave them.
template <typename T, int NT, int NS, int NP, int CW>
__global__ void __launch_bounds__(terms_threads(CW), 1)
gram_umma_f32_kernel(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_r,
                     const F32Params p, float *__restrict__ partials, double *__restrict__ bpart,
                     int *__restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages];     // stage s holds a landed tile
  __shared__ __align__(8) uint64_t bar_empty[kMaxStages];    // ... has been converted
  __shared__ __align__(8) uint64_t bar_op_full[kMaxOps];     // operand buffer o holds the terms of a block
  __shared__ __align__(8) uint64_t bar_op_empty[kMaxOps];    // ... has been read by its MMAs
  __shared__ __align__(8) uint64_t bar_acc_full[2];
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ uint32_t tmem_base_sh;
  constexpr uint32_t ES = (uint32_t)sizeof(T);
  constexpr int kConvWarps = CW, kConvThreads = 32 * CW, kConvRows = terms_conv_rows(CW), kThreads = terms_threads(CW);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = p.m;
  const int scols = p.nsub * kBlockCols;
  const int rows8 = (2 * m + 7) & ~7;                                      // rows a stage holds (8-row boxes)
  const uint32_t rows_bytes = (uint32_t)rows8 * scols * ES;
  const uint32_t stage_bytes = rows_bytes + (uint32_t)scols * 4u;          // the rows, then the piece of r (fp32)
  const int op_rows = p.npad > 128 ? p.npad : 128;                         // operand A spans 128 rows
  const uint32_t op_bytes = (uint32_t)op_rows * 128u;
  const uint32_t ops_base = (smem_u32(smem_raw) + 1023u) & ~1023u;         // swizzle atoms need 1024-B alignment
  uint8_t *ops_ptr = smem_raw + (ops_base - smem_u32(smem_raw));
  const uint32_t stages_base = ops_base + (uint32_t)p.nops * op_bytes;
  uint8_t *stages_ptr = ops_ptr + (size_t)p.nops * op_bytes;

  const long long blk_lo = p.nblk * (long long)blockIdx.x / gridDim.x;
  const long long blk_hi = p.nblk * (long long)(blockIdx.x + 1) / gridDim.x;
  const int nsb = (int)(blk_hi - blk_lo);                                  // 64-column blocks of this CTA
  const int n_iter = (nsb + p.nsub - 1) / p.nsub;                          // stages it streams

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), kConvWarps);
    }
    for (int o = 0; o < p.nops; ++o) {
      mbar_init(smem_u32(&bar_op_full[o]), kConvWarps);
      mbar_init(smem_u32(&bar_op_empty[o]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_acc_full[b]), 1);
      mbar_init(smem_u32(&bar_acc_empty[b]), kDrainWarps);
    }
    mbar_init_fence();
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_g) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_r) : "memory");
  }
  // operand rows no converter ever writes (past the NT m term rows) are zeroed once
  for (int o = 0; o < p.nops; ++o) {
    uint8_t *z = ops_ptr + (size_t)o * op_bytes + (size_t)(NT * m) * 128;   // whole rows: 128 B each, swizzle-neutral
    const uint32_t nbytes = (uint32_t)(op_rows - NT * m) * 128u;
    for (uint32_t off = threadIdx.x * 16; off < nbytes; off += kThreads * 16)
      *reinterpret_cast<uint4 *>(z + off) = make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_sh)), "r"(512u) : "memory");   // two accumulators of 256 columns
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_sh;
  cdg_grid_dep_wait();            // r is written by the launch before this one
  const long long deadline = clock64() + kCdgWaitCycles;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const int nbox = rows8 >> 3;
      const uint32_t box_bytes = 8u * scols * ES;
      int issued = 0;
      bool ok = true;
      int s = 0;
      uint32_t turn = 0;
      for (int it = 0; it < n_iter; ++it) {
        if (turn > 0) ok = f32_wait(smem_u32(&bar_empty[s]), (turn - 1) & 1, deadline);
        if (!ok) break;
        const int col = (int)((blk_lo + (long long)it * p.nsub) * kBlockCols);   // a multiple of 64 floats
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t dst = stages_base + (uint32_t)s * stage_bytes;
        mbar_expect_tx(full, stage_bytes);
        for (int q = 0; q < nbox; ++q) tma_load_2d(dst + q * box_bytes, &tm_g, col, q * 8, full);
        tma_load_2d(dst + nbox * box_bytes, &tm_r, col, 0, full);
        issued = it + 1;
        if (++s == p.stages) { s = 0; ++turn; }
      }
      if (!ok) {
        atomicOr(status, CDG_ST_TIMEOUT);
        for (int it = max(0, issued - p.stages); it < issued; ++it)
          f32_wait(smem_u32(&bar_full[it % p.stages]), (it / p.stages) & 1, clock64() + kCdgWaitCycles);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: the warp loops converged, an elected lane issues ----------------
    // kind::f16, D = f32, A = B = bf16, both K-major, M = 128 (64 when A has at most 64 rows), N = npad
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)p.npad >> 3) << 17) | (((uint32_t)p.mma_m >> 4) << 24);
    bool ok = true;
    int o = 0, c = 0, in_chunk = 0;
    uint32_t op_parity = 0;
    for (int g = 0; g < nsb; ++g) {
      const int buf = c & 1;
      const bool chunk_start = in_chunk == 0;
      if (chunk_start && c >= 2) ok = f32_wait(smem_u32(&bar_acc_empty[buf]), ((c >> 1) - 1) & 1, deadline);
      if (ok) ok = f32_wait(smem_u32(&bar_op_full[o]), op_parity, deadline);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t acc = tmem_acc + (uint32_t)buf * 256u;
      const uint64_t desc = f32_umma_desc(ops_base + (uint32_t)o * op_bytes);
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const uint64_t dk = desc + (uint64_t)(k4 * 2);     // 16 bf16 = 32 bytes further along K
        if (f32_elect_one()) f32_umma(acc, dk, dk, idesc, !(chunk_start && k4 == 0));
      }
      const bool chunk_end = (in_chunk == p.drain - 1) || (g == nsb - 1);
      if (f32_elect_one()) {
        f32_commit(smem_u32(&bar_op_empty[o]));
        if (chunk_end) f32_commit(smem_u32(&bar_acc_full[buf]));
      }
      if (++in_chunk == p.drain) { in_chunk = 0; ++c; }
      if (++o == p.nops) { o = 0; op_parity ^= 1u; }
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
  } else if (warp < 2 + kConvWarps) {
    // ---------------- converters: tile -> differences -> NT bf16 terms; b on the side ----------------
    const int ct = threadIdx.x - 64;                 // 0..191
    const int q = ct & 15;                           // this thread's 4 columns of every row it takes
    const int row0 = ct >> 4;                        // rows row0, row0 + 12, ... of a pass
    // Byte offsets that never change (pass 0): of the thread's 4 columns inside a stage (block 0)
    // and of its 8 bytes of term t inside an operand buffer -- row t m + i, 128 B per row, 16-byte
    // chunk (q >> 1) at chunk (q >> 1) ^ (row & 7), upper half of the chunk for odd q.  A further
    // pass lies pass_rows rows on: a multiple of 8, so the swizzle phase of every row is the same.
    uint32_t src[NS], dst[NT][NS];
#pragma unroll
    for (int j = 0; j < NS; ++j) {
      const int i = row0 + kConvRows * j;
      src[j] = (uint32_t)(i * scols + q * 4) * ES;
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        const int row = t * m + i;
        dst[t][j] = (uint32_t)(row * 128 + ((((q >> 1) ^ (row & 7)) << 4) | ((q & 1) << 3)));
      }
    }
    const uint32_t z2_off = (uint32_t)(m * scols) * ES;          // from a row of slab 0 to its partner in slab 1
    const uint32_t pass_src = (uint32_t)(p.pass_rows * scols) * ES, pass_dst = (uint32_t)p.pass_rows * 128u;
    float bacc[NP][NS];
    double bsum[NP][NS];
#pragma unroll
    for (int hp = 0; hp < NP; ++hp)
#pragma unroll
      for (int j = 0; j < NS; ++j) { bacc[hp][j] = 0.f; bsum[hp][j] = 0.0; }
    bool ok = true;
    int s = 0, o = 0, since_flush = 0;
    uint32_t full_parity = 0, turn_o = 0;
    for (int it = 0; it < n_iter && ok; ++it) {
      ok = __all_sync(0xffffffffu, f32_wait(smem_u32(&bar_full[s]), full_parity, deadline));   // the lanes leave together
      if (!ok) break;
      const uint8_t *tile = stages_ptr + (size_t)s * stage_bytes;
      const float *rt = reinterpret_cast<const float *>(tile + rows_bytes);
      const int cnt = min(p.nsub, nsb - it * p.nsub);      // blocks past the range belong to the next CTA
      for (int sub = 0; sub < cnt; ++sub) {
        if (turn_o > 0) ok = __all_sync(0xffffffffu, f32_wait(smem_u32(&bar_op_empty[o]), (turn_o - 1) & 1, deadline));
        if (!ok) break;
        uint8_t *op = ops_ptr + (size_t)o * op_bytes;
        const float4 rv = *reinterpret_cast<const float4 *>(rt + sub * kBlockCols + q * 4);
#pragma unroll
        for (int hp = 0; hp < NP; ++hp) {
          // Straight-line code from the loads to the stores: every load first, then the split one
          // step at a time over all slots (each step's 2 NS operations are independent of one another).
          uint32_t vmask = 0;
          float c[NS][4];
#pragma unroll
          for (int j = 0; j < NS; ++j) {
            int i = hp * p.pass_rows + row0 + kConvRows * j;
            const bool in_pass = row0 + kConvRows * j < p.pass_rows;
            if (i < m && in_pass) vmask |= 1u << j;
            // a slot past the last row loads a valid row (row 0 of the pass) and stores nothing
            const uint32_t so = (i < m && in_pass) ? src[j] : (uint32_t)(q * 4) * ES;
            float za[4], zb[4];
            TermIn<T>::ld(tile + hp * pass_src + so + sub * (kBlockCols * ES), za);
            TermIn<T>::ld(tile + hp * pass_src + so + z2_off + sub * (kBlockCols * ES), zb);
#pragma unroll
            for (int e = 0; e < 4; ++e) c[j][e] = za[e] - zb[e];
          }
          uint32_t term[NT][NS][2];
          float r1[NS][4];
#pragma unroll
          for (int j = 0; j < NS; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) r1[j][e] = c[j][e];
#pragma unroll
          for (int t = 0; t < NT; ++t) {
#pragma unroll
            for (int j = 0; j < NS; ++j)
#pragma unroll
              for (int h = 0; h < 2; ++h) term[t][j][h] = pack_bf16x2(r1[j][2 * h], r1[j][2 * h + 1]);
            if (t + 1 < NT) {
#pragma unroll
              for (int j = 0; j < NS; ++j)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                  r1[j][2 * h] -= __uint_as_float(term[t][j][h] << 16);
                  r1[j][2 * h + 1] -= __uint_as_float(term[t][j][h] & 0xffff0000u);
                }
            }
          }
#pragma unroll
          for (int j = 0; j < NS; ++j) {
            float t = fmaf(rv.x, c[j][0], bacc[hp][j]);
            t = fmaf(rv.y, c[j][1], t);
            t = fmaf(rv.z, c[j][2], t);
            t = fmaf(rv.w, c[j][3], t);
            bacc[hp][j] = (vmask & (1u << j)) ? t : 0.f;
          }
#pragma unroll
          for (int j = 0; j < NS; ++j) {
            if (vmask & (1u << j)) {
#pragma unroll
              for (int t = 0; t < NT; ++t)
                *reinterpret_cast<uint2 *>(op + hp * pass_dst + dst[t][j]) = make_uint2(term[t][j][0], term[t][j][1]);
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMA reads these bytes through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_op_full[o]));
        if (++o == p.nops) { o = 0; ++turn_o; }
        if (++since_flush == kFlushBlocks) {
          since_flush = 0;
#pragma unroll
          for (int hp = 0; hp < NP; ++hp)
#pragma unroll
            for (int j = 0; j < NS; ++j) { bsum[hp][j] += (double)bacc[hp][j]; bacc[hp][j] = 0.f; }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_empty[s]));
      if (++s == p.stages) { s = 0; full_parity ^= 1u; }
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
    // the ring of stages is idle now (every tile has landed and been converted): it holds the
    // per-thread sums of b while the 16 threads that shared a row are added up, in q order
    asm volatile("bar.sync 2, %0;" ::"r"(kConvThreads) : "memory");        // the converter warps only
    double *bred = reinterpret_cast<double *>(stages_ptr);
    if (ok) {
#pragma unroll
      for (int hp = 0; hp < NP; ++hp)
#pragma unroll
        for (int j = 0; j < NS; ++j) bred[(ct * NP + hp) * NS + j] = bsum[hp][j] + (double)bacc[hp][j];
    }
    asm volatile("bar.sync 2, %0;" ::"r"(kConvThreads) : "memory");
    if (ct < m && ok) {
      const int hp = ct / p.pass_rows, within = ct % p.pass_rows;
      const int t0 = (within % kConvRows) * 16, j = within / kConvRows;
      double v = 0.0;
#pragma unroll
      for (int qq = 0; qq < 16; ++qq) v += bred[((t0 + qq) * NP + hp) * NS + j];
      bpart[(size_t)blockIdx.x * kMaxM + ct] = v;
    }
  } else {
    // ---------------- accumulator read-back: TMEM chunks -> partial D ----------------
    const int dw = warp - (2 + kConvWarps);          // 0..7
    const int lg = warp & 3;                         // TMEM lane group this warp may read; four consecutive warps cover all four
    const int half = dw >> 2;                        // pieces of 16 columns: this warp takes piece 2 pp + half
    // M = 128: row r of D lies in TMEM lane r.  M = 64: in lane 32 (r / 16) + r % 16, the first 16
    // lanes of each lane group (the other lanes hold nothing of this product: row 128 = none).
    int row = lg * 32 + lane;
    if (p.mma_m == 64) row = (lane < 16) ? lg * 16 + lane : 128;
    const int nchunks = (nsb + p.drain - 1) / p.drain;
    const int rows_needed = (NT == 3) ? 2 * m : m;   // rows of D the combine reads
    float *dst = partials + ((size_t)blockIdx.x * 128 + (row & 127)) * (size_t)p.npad;
    // NT == 3 (N <= 192): the chunks are added in fp32 registers and stored once.  NT == 2
    // (N <= 256): each chunk is added to the partial in global memory (first chunk: stored).
    constexpr int kPieces = (NT == 3) ? 6 : 8;       // pieces of 16 columns per warp
    float accr[(NT == 3) ? kPieces * 16 : 1];
    if constexpr (NT == 3) {
#pragma unroll
      for (int j = 0; j < kPieces * 16; ++j) accr[j] = 0.f;
    }
    bool ok = true;
    for (int c = 0; c < nchunks && ok; ++c) {
      const int buf = c & 1;
      ok = __all_sync(0xffffffffu, f32_wait(smem_u32(&bar_acc_full[buf]), (c >> 1) & 1, deadline));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int pp = 0; pp < kPieces; ++pp) {
        const int piece = 2 * pp + half;
        if (piece * 16 < p.npad) {
          uint32_t v[16];
          const uint32_t taddr = tmem_acc + (uint32_t)buf * 256u + ((uint32_t)(lg * 32) << 16) + (uint32_t)(piece * 16);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
              "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
                "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
                "=r"(v[14]), "=r"(v[15])
              : "r"(taddr) : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if constexpr (NT == 3) {
#pragma unroll
            for (int j = 0; j < 16; ++j) accr[pp * 16 + j] += __uint_as_float(v[j]);
          } else if (row < rows_needed) {
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
              float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (c > 0) acc4 = *reinterpret_cast<const float4 *>(dst + piece * 16 + j);   // this thread's own earlier store
              acc4.x += __uint_as_float(v[j]); acc4.y += __uint_as_float(v[j + 1]);
              acc4.z += __uint_as_float(v[j + 2]); acc4.w += __uint_as_float(v[j + 3]);
              *reinterpret_cast<float4 *>(dst + piece * 16 + j) = acc4;
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
    if constexpr (NT == 3) {
      if (row < rows_needed) {
#pragma unroll
        for (int pp = 0; pp < kPieces; ++pp) {
          const int piece = 2 * pp + half;
          if (piece * 16 < p.npad) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              *reinterpret_cast<float4 *>(dst + piece * 16 + j) =
                  make_float4(accr[pp * 16 + j], accr[pp * 16 + j + 1], accr[pp * 16 + j + 2], accr[pp * 16 + j + 3]);
          }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(512u) : "memory");
  }
}

// Sum of the per-CTA partial D over the CTAs, in index order, in fp64: block a adds row a
// (its columns x 3 ranges of CTAs, the range sums then added in range order) and, for a < m,
// b_a.  The block that takes the last ticket forms G from the summed rows (the term products
// listed at the top of this file), writes (G, b) and takes the step's decisions.
constexpr int kCombThreads = 768;
constexpr int kCombRanges = kCombThreads / kMaxN;    // 3
__global__ void __launch_bounds__(kCombThreads)
umma_f32_combine_kernel(const float *__restrict__ partials, const double *__restrict__ bpart, int ctas, int npad,
                        int m, int nt, double *__restrict__ dsum, double *__restrict__ gram, int *__restrict__ status,
                        const CdgTail tail) {
  extern __shared__ double scan_sh[];              // (4m + m*m) doubles: the scan's arrays and G
  __shared__ double part[kCombRanges][kMaxN];
  __shared__ int is_last;
  cdg_grid_dep_wait();            // the partials come from the launch before this one
  const int a = blockIdx.x;
  const int col = threadIdx.x % kMaxN, qr = threadIdx.x / kMaxN;
  if (col < npad) {
    const int c_lo = ctas * qr / kCombRanges, c_hi = ctas * (qr + 1) / kCombRanges;
    const float *P = partials + (size_t)a * npad + col;
    const size_t cs = (size_t)128 * npad;
    double v = 0.0;
    int c = c_lo;
    for (; c + 8 <= c_hi; c += 8) {
      float x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = P[(size_t)(c + u) * cs];
#pragma unroll
      for (int u = 0; u < 8; ++u) v += (double)x[u];
    }
    for (; c < c_hi; ++c) v += (double)P[(size_t)c * cs];
    part[qr][col] = v;
  }
  __syncthreads();
  if (threadIdx.x < npad)
    dsum[(size_t)a * kMaxN + threadIdx.x] = (part[0][threadIdx.x] + part[1][threadIdx.x]) + part[2][threadIdx.x];
  if (a < m && threadIdx.x >= kCombThreads - 32) {
    // b_a: lane l adds the CTAs l, l + 32, ... in that order, then a fixed butterfly
    const int lane = threadIdx.x & 31;
    double v = 0.0;
    for (int c = lane; c < ctas; c += 32) v += bpart[(size_t)c * kMaxM + a];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    if (lane == 0) gram[(size_t)m * m + a] = v;
  }

  // ---- the block that takes the last ticket has every summed row before it ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(tail.ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const ScanSmem S = scan_smem(scan_sh, m);
  // four entries per thread and round, every load of the round in flight before the first sum
  for (int e0 = threadIdx.x; e0 < m * m; e0 += 4 * kCombThreads) {
    double x[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * kCombThreads;
      if (e < m * m) {
        const int k = e / m, i = e % m;
        const double *Dk = dsum + (size_t)k * kMaxN;
        if (nt == 3) {
          const double *Dmk = dsum + (size_t)(m + k) * kMaxN;
          x[u][0] = __ldcg(Dk + i); x[u][1] = __ldcg(Dk + m + i); x[u][2] = __ldcg(Dk + 2 * m + i);      // hh hm hl
          x[u][3] = __ldcg(Dmk + i); x[u][4] = __ldcg(Dmk + m + i); x[u][5] = __ldcg(Dmk + 2 * m + i);   // mh mm ml
          x[u][6] = __ldcg(dsum + (size_t)i * kMaxN + 2 * m + k);                                        // lh
          x[u][7] = __ldcg(dsum + (size_t)(m + i) * kMaxN + 2 * m + k);                                  // lm
        } else {
          x[u][0] = __ldcg(Dk + i); x[u][1] = __ldcg(Dk + m + i);                                        // hh hl
          x[u][2] = __ldcg(dsum + (size_t)i * kMaxN + m + k);                                            // lh
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * kCombThreads;
      if (e < m * m) {
        // smallest terms first
        const double v = (nt == 3) ? ((((x[u][5] + x[u][7]) + (x[u][2] + x[u][6])) + x[u][4]) + (x[u][1] + x[u][3])) + x[u][0]
                                   : (x[u][1] + x[u][2]) + x[u][0];
        S.g[e] = v;
        gram[e] = v;
      }
    }
  }
  for (int j = threadIdx.x; j < m; j += kCombThreads) S.t[j] = __ldcg(gram + (size_t)m * m + j);
  if (threadIdx.x == 0) *tail.ticket = 0u;                    // ready for the next launch
  if (!tail.enabled) return;
  scan_load_pairs(S, tail.perm_cur, m, tail.n, tail.k);
  __syncthreads();
  scan_decide_and_write<4>(S, S.g, m, tail.n, tail.k, tail.perm_next, tail.signs, tail.margins, tail.rnorm2, status,
                           tail.rule);
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D map over `rows` rows of d columns of fp32 or bf16, box [box_rows][cols], no swizzle; columns
// past d read as zeros
bool encode_rows(CUtensorMap *map, const void *base, long long d, int rows, int box_rows, int cols, int elem_bytes) {
  EncodeFn fn = (EncodeFn)cdg_tensor_map_encoder();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int NT, int NS, int NP, int CW = 6>
cudaError_t terms_launch(cdgrab_ctx *h, const CUtensorMap &tm_g, const F32Params &p, cudaStream_t st) {
  return cdg_launch_dep(h, gram_umma_f32_kernel<T, NT, NS, NP, CW>, dim3(h->f32_ctas), dim3(terms_threads(CW)), h->f32_smem,
                        st, tm_g, h->tm_f32r, p, h->umma_partials, h->f32_bpart, h->status);
}

cudaError_t terms_open_limits() {
  cudaError_t e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 1, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 2, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 3, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 4, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 5, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 6, 1, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<__nv_bfloat16, 2, 4, 2, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<__nv_bfloat16, 2, 5, 2, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<__nv_bfloat16, 2, 6, 2, 6>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<float, 3, 4, 1, 8>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(gram_umma_f32_kernel<__nv_bfloat16, 2, 4, 2, 8>);
  if (e == cudaSuccess) e = cdg_open_smem_limit(umma_f32_combine_kernel);
  return e;
}

// bf16 gradients: 65..128 workers take two converter passes of pass_rows rows each
inline int bf16_pass_rows(int m) { return (((m + 1) / 2) + 7) & ~7; }

}  // namespace

// fp32: rows whose pitch is a multiple of 16 bytes; 2m <= 128 rows of hi and mid terms fill the MMA's M.
// bf16: 65 <= m <= 128 (up to 64 workers the raw rows go through the MMA as they lie in HBM).
bool cdg_umma_f32_supported(int m, long long d) {
  return m >= 1 && m <= 64 && d % 4 == 0 && d >= 4096 && d < (1ll << 31) - 512 && cdg_tensor_map_encoder() != nullptr;
}
bool cdg_umma_terms_bf16_supported(int m, long long d) {
  return m > 64 && m <= kMaxM && d % 8 == 0 && d >= 4096 && d < (1ll << 31) - 512 && cdg_tensor_map_encoder() != nullptr;
}

int cdg_umma_f32_setup(cdgrab_ctx *h) {
  const int m = h->m;
  const int nt = (h->dtype == CDGRAB_F32) ? 3 : 2;
  const size_t es = (h->dtype == CDGRAB_F32) ? 4 : 2;
  h->f32_nt = nt;
  h->f32_npad = ((nt * m + 15) / 16) * 16;
  const int rows8 = (2 * m + 7) & ~7;
  const int op_rows = h->f32_npad > 128 ? h->f32_npad : 128;
  const size_t op_bytes = (size_t)op_rows * 128;
  // stage width: 128 columns (512 or 256 contiguous bytes per row and copy) while two such stages fit
  // beside the operand buffers (three, or two when three leave no room), else 64;
  // CDGRAB_F32_NSUB / CDGRAB_F32_NOPS override
  int nsub = 2, nops = 3;
  bool nops_forced = false;
  if (const char *e = getenv("CDGRAB_F32_NSUB")) {
    const int v = atoi(e);
    if (v == 1 || v == 2 || v == 4) nsub = v;
  }
  if (const char *e = getenv("CDGRAB_F32_NOPS")) {
    const int v = atoi(e);
    if (v >= 2 && v <= kMaxOps) { nops = v; nops_forced = true; }
  }
  const size_t budget = (size_t)kCdgMaxDynSmem - 1024 - 4 * 1024;   // static shared memory: the barriers
  auto stage_of = [&](int ns) { return (size_t)rows8 * ns * kBlockCols * es + (size_t)ns * kBlockCols * 4; };
  size_t stage_bytes = stage_of(nsub);
  if (!nops_forced && nops > 2 && budget < nops * op_bytes + 2 * stage_bytes) nops = 2;
  while (nsub > 1 && budget < nops * op_bytes + 2 * stage_bytes) {
    nsub >>= 1;
    stage_bytes = stage_of(nsub);
  }
  if (budget < nops * op_bytes + 2 * stage_bytes) return CDGRAB_ERR_INVALID;
  int stages = (int)((budget - nops * op_bytes) / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (const char *e = getenv("CDGRAB_F32_STAGES")) {
    const int v = atoi(e);
    if (v >= 2 && v < stages) stages = v;
  }
  if (stages < 2) return CDGRAB_ERR_INVALID;
  h->f32_nsub = nsub;
  h->f32_nops = nops;
  h->f32_stages = stages;
  h->f32_smem = 1024 + nops * op_bytes + stages * stage_bytes;
  // TMEM chunk: about 512 columns for fp32 inputs (held to the 1e-6 sign tolerance), 4096 for bf16;
  // CDGRAB_UMMA_DRAIN overrides
  h->f32_drain = (nt == 3 ? 512 : 4096) / kBlockCols;
  if (const char *e = getenv("CDGRAB_UMMA_DRAIN")) {
    const int v = atoi(e);
    if (v >= 1 && v <= (1 << 20)) h->f32_drain = v;
  }
  const long long nblk = (h->d + kBlockCols - 1) / kBlockCols;
  h->f32_ctas = (int)(nblk < h->num_sms ? nblk : h->num_sms);
  const size_t pbytes = sizeof(float) * 128 * (size_t)h->f32_npad * h->f32_ctas;
  if (cdg_alloc(h, &h->umma_partials, pbytes) != cudaSuccess ||
      cdg_alloc(h, &h->f32_bpart, sizeof(double) * kMaxM * (size_t)h->f32_ctas) != cudaSuccess ||
      cdg_alloc(h, &h->f32_dsum, sizeof(double) * 128 * kMaxN) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_NOMEM;
  }
  if (cudaMemset(h->umma_partials, 0, pbytes) != cudaSuccess ||
      cudaMemset(h->f32_bpart, 0, sizeof(double) * kMaxM * (size_t)h->f32_ctas) != cudaSuccess ||
      cudaMemset(h->f32_dsum, 0, sizeof(double) * 128 * kMaxN) != cudaSuccess)
    return CDGRAB_ERR_CUDA;
  if (!encode_rows(&h->tm_f32r, h->r, h->d, 1, 1, nsub * kBlockCols, 4)) return CDGRAB_ERR_CUDA;
  if (terms_open_limits() != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  h->umma_fused = h->shard ? 0 : 1;      // a shard's decisions wait for the sum over shards
  if (const char *e = getenv("CDGRAB_UMMA_FUSE_TAIL")) {
    if (atoi(e) == 0) h->umma_fused = 0;
  }
  // fp32 with at most 32 workers: hi and mid terms are 2m <= 64 rows, so M = 64 reads half the A
  // bytes per MMA (pass 1 is bound by shared-memory bandwidth there: 4 % faster at m = 32);
  // CDGRAB_F32_M64=0 keeps M = 128
  h->f32_mma_m = (nt == 3 && 2 * m <= 64) ? 64 : 128;
  if (const char *e = getenv("CDGRAB_F32_M64")) {
    if (atoi(e) == 0) h->f32_mma_m = 128;
  }
  h->f32_conv8 = 1;                      // CDGRAB_F32_CONV8=0: six converter warps at every size
  if (const char *e = getenv("CDGRAB_F32_CONV8")) h->f32_conv8 = atoi(e) ? 1 : 0;
  h->umma_f32 = 1;
  return CDGRAB_OK;
}

void cdg_umma_f32_teardown(cdgrab_ctx *h) {
  cdg_free(h->f32_bpart);
  cdg_free(h->f32_dsum);
  h->f32_bpart = nullptr;
  h->f32_dsum = nullptr;
}

cudaError_t cdg_launch_gram_umma_f32(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  const int es = (h->dtype == CDGRAB_F32) ? 4 : 2;
  int slot = h->tm_f32g.find(grads);
  if (slot < 0) {
    slot = h->tm_f32g.victim();
    if (!encode_rows(&h->tm_f32g.maps[slot][0], grads, h->d, 2 * h->m, 8, h->f32_nsub * kBlockCols, es))
      return cudaErrorInvalidValue;
    h->tm_f32g.commit(slot, grads);
  }
  F32Params p;
  p.m = h->m;
  p.npad = h->f32_npad;
  p.nsub = h->f32_nsub;
  p.stages = h->f32_stages;
  p.nops = h->f32_nops;
  p.drain = h->f32_drain;
  p.nblk = (h->d + kBlockCols - 1) / kBlockCols;
  p.mma_m = h->f32_mma_m;
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    const CUtensorMap &tm = h->tm_f32g.maps[slot][0];
    // rows per converter thread and pass: up to 5 with six converter warps; where they would take 6, eight warps take 4
    if (h->f32_nt == 3) {
      p.pass_rows = (h->m + 7) & ~7;
      const int ns = (h->m + terms_conv_rows(6) - 1) / terms_conv_rows(6);
      if (ns > 5 && h->f32_conv8) {
        terms_launch<float, 3, 4, 1, 8>(h, tm, p, st);
      } else switch (ns) {
        case 1: terms_launch<float, 3, 1, 1>(h, tm, p, st); break;
        case 2: terms_launch<float, 3, 2, 1>(h, tm, p, st); break;
        case 3: terms_launch<float, 3, 3, 1>(h, tm, p, st); break;
        case 4: terms_launch<float, 3, 4, 1>(h, tm, p, st); break;
        case 5: terms_launch<float, 3, 5, 1>(h, tm, p, st); break;
        default: terms_launch<float, 3, 6, 1>(h, tm, p, st); break;
      }
    } else {
      p.pass_rows = bf16_pass_rows(h->m);                      // 40..64
      const int ns = (p.pass_rows + terms_conv_rows(6) - 1) / terms_conv_rows(6);
      if (ns > 5 && h->f32_conv8) {
        terms_launch<__nv_bfloat16, 2, 4, 2, 8>(h, tm, p, st);
      } else switch (ns) {
        case 4: terms_launch<__nv_bfloat16, 2, 4, 2>(h, tm, p, st); break;
        case 5: terms_launch<__nv_bfloat16, 2, 5, 2>(h, tm, p, st); break;
        default: terms_launch<__nv_bfloat16, 2, 6, 2>(h, tm, p, st); break;
      }
    }
  }
  {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    const int rows = (h->f32_nt == 3) ? 2 * h->m : h->m;
    cdg_launch_dep(h, umma_f32_combine_kernel, dim3(rows), dim3(kCombThreads), scan_smem_bytes(h->m, true), st,
                   (const float *)h->umma_partials, (const double *)h->f32_bpart, h->f32_ctas, h->f32_npad, h->m,
                   h->f32_nt, h->f32_dsum, h->gram, h->status, cdg_tail_of(h, h->umma_fused));
  }
  return cudaGetLastError();
}
