// Pass 1 on the 5th-generation tensor cores (tcgen05) for bf16 gradients, m <= 64.
//
// The 2m gradient rows of a step ([2][m][d], K-major exactly as they lie in HBM) are the
// operand A of  H = A A^T  (2m x 2m); every bf16 x bf16 product is exact in the fp32
// accumulator, so no difference has to be rounded to bf16.  The Gram matrix of the pair
// differences c_i = z1_i - z2_i follows afterwards in fp64:
//     G_ki = H[k][i] - H[k][m+i] - H[m+k][i] + H[m+k][m+i].
// The running sum r (fp32) goes in as three bf16 rows hi + mid + lo = r exactly (3 x 8
// significand bits) appended to operand B, so
//     b_i = <r, c_i> = sum_j (H[i][R+j] - H[m+i][R+j])
// falls out of the same MMA.  The rows are formed inside the kernel: the TMA brings the fp32
// piece of r of a stage (4 bytes per column), a converter warp splits it and writes the three
// rows into the stage's r row group in the swizzled layout the TMA would have produced.
// (CDGRAB_UMMA_RCONV=0: pass 2 keeps a bf16 copy [3][d] of r in HBM and the TMA brings its rows;
// 12 instead of 4 bytes of r traffic per column and step on top of pass 2's own 8.)
//
// One persistent CTA per SM owns a contiguous K range (split-K) in blocks of 64 columns.
// A pipeline stage holds `subs` consecutive blocks.  Rows are loaded in groups of 8: a TMA box
// {64 columns, 8 rows, subs blocks} touches only 8 rows and subs*128 contiguous bytes of each,
// which keeps address translation and DRAM pages local even though consecutive rows lie
// hundreds of megabytes apart; a 4-D map {64 columns, 8 rows, blocks, groups} brings all full
// groups of a stage with one instruction in the same order.  In shared memory a stage is
// [row group][block][8 rows][128 B, 128-byte swizzle]; the MMA descriptors walk row groups
// with a stride of subs*1024 bytes.  Row groups 0..box_rows/8-1 hold gradient rows (rows past
// 2m are zero-filled by TMA), the next group holds the three r rows, and one more group of
// zeros (written once) pads N to a multiple of 16.  The same bytes serve as operand A (16
// row groups from the block base) and operand B (the first N = box_rows + 16 rows).  A ragged
// last block (d not a multiple of 64) is loaded with 2-D boxes of 8 rows into the same layout.
// With 2m <= 64 one MMA takes two blocks at once (N = 160; layout at the top of the kernel).
// Roles: warp 0 TMA producer, warp 1 MMA issuer (the warp loops converged, an elected lane
// issues) and TMEM owner, warps 2..5 drain the accumulator (tcgen05.ld) chunk by chunk into
// fp32 registers and write the CTA's partial H, warp 6 converts r.  The combine kernel's last block also takes the
// step's decisions.
// Every wait is bounded: on expiry the CTA raises the time-out bit of the status word,
// drains the copies it has in flight, frees its TMEM and returns.
#include <cudaTypedefs.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "ptx.cuh"
#include "scan.cuh"

namespace {

constexpr int kThreads = 224;           // TMA producer, MMA issuer, four read-back warps, one converter of r
constexpr int kMaxStages = 8;
constexpr int kSubCols = 64;             // bf16 columns per TMA box = one 128-byte swizzle row
constexpr int kRBoxRows = 16;
constexpr int kMaxCols = 144;            // MMA N at m = 64: 128 gradient rows + 16
constexpr long long kWaitCycles = kCdgWaitCycles;

struct UmmaParams {
  int box_rows;        // gradient rows held per block (2m rounded up to 16; 64 when paired)
  int ncols;           // columns of a partial H row = box_rows + 16 (MMA N, or half of it when paired)
  int rows_used;       // 2m
  int subs;            // 64-column blocks per stage
  int stages;
  long long nblk_full; // d / 64: blocks loaded by the 3-D maps
  int tail;            // 1 when d % 64 != 0: one more, ragged block
  int drain;           // pipeline iterations accumulated in TMEM before the sum is drained
  int g4;              // full 8-row groups fetched by one 4-D copy (0: per-group copies only)
  int paired;          // 2m <= 64: blocks j and j + subs/2 of a stage share one MMA (see the kernel)
  int rconv;           // 1: r arrives as fp32 and warp 6 writes its three bf16 rows; 0: the rows come from HBM
  int rbox;            // 64-column blocks of r per fp32 copy (a divisor of the blocks per (half) stage, at most 4)
};

// K-major, 128-byte swizzle: rows 128 B apart, 8-row groups `sbo` bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for this layout)
  d |= (uint64_t)(sbo >> 4) << 32;                 // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version
  d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
  return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accum) : "memory");
}
// true in exactly one lane of a converged warp (the same lane every time)
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
gram_umma_kernel(const __grid_constant__ CUtensorMap tm_g3, const __grid_constant__ CUtensorMap tm_r3,
                 const __grid_constant__ CUtensorMap tm_g2, const __grid_constant__ CUtensorMap tm_r2,
                 const __grid_constant__ CUtensorMap tm_g4, const __grid_constant__ CUtensorMap tm_r32,
                 const UmmaParams p, float *__restrict__ partials, int *__restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
  __shared__ __align__(8) uint64_t bar_r32[kMaxStages];   // the fp32 piece of r of stage s has landed (rconv)
  __shared__ __align__(8) uint64_t bar_conv[kMaxStages];  // ... and its bf16 rows are written
  __shared__ __align__(8) uint64_t bar_acc_full[2];    // accumulator buffer b holds a finished chunk
  __shared__ __align__(8) uint64_t bar_acc_empty[2];   // ... has been read back and may be overwritten
  __shared__ uint32_t tmem_base_sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-B alignment
  // Paired mode (2m <= 64).  With at most 64 gradient rows, half of a 128-row MMA would idle
  // and the issue rate of the small MMAs, not HBM, would bound the kernel.  So one MMA takes two
  // 64-column blocks at once: a stage is laid out as 20 row groups
  //   [0..7] rows of block j | [8..15] rows of block j + subs/2 | [16] r of j | [17] 0 | [18] r of j' | [19] 0
  // A = groups 0..15 (M = 128), B = all 20 (N = 160).  D rows 0..63 x columns 0..63 and 128..143
  // hold block j's products, rows 64..127 x columns 64..127 and 144..159 block j''s; the other
  // entries are cross terms nobody reads.
  // When the r rows are written by the converter warp (rconv), both blocks' rows share group 16
  // (rows 0..2 r of j, rows 3..5 r of j') and group 17 is the zero padding: 18 groups, N = 144,
  // block j's b in columns 128..130 of rows 0..63 and block j''s in columns 131..133 of rows 64..127.
  const int paired = p.paired;
  const int hb = p.subs >> 1;                                    // blocks per half stage (paired)
  const uint32_t group_bytes = (uint32_t)(paired ? hb : p.subs) * 1024u;   // one row group of a stage
  const int ngroups = paired ? (p.rconv ? 18 : 20) : (p.ncols >> 3);
  const int ggroups = p.box_rows >> 3;                           // gradient row groups
  const uint32_t stage_bytes = group_bytes * ngroups;
  // rconv: the fp32 pieces of r (256 bytes per block, subs blocks per stage) lie behind the
  // stages and the slack operand A may read past the last stage
  const int rconv = p.rconv;
  const uint32_t r32_off = (uint32_t)p.stages * stage_bytes + (ngroups < 16 ? (uint32_t)(16 - ngroups) * group_bytes : 0u);

  // this CTA's K range in full blocks; the last CTA also owns the ragged block, taken first.
  // Paired: whole stages per CTA, so that both halves of a stage belong to the same CTA (blocks
  // past the end of the rows are read as zeros).
  long long blk_lo, blk_hi;
  if (paired) {
    const long long units = (p.nblk_full + p.subs - 1) / p.subs;
    blk_lo = units * (long long)blockIdx.x / gridDim.x * p.subs;
    blk_hi = units * (long long)(blockIdx.x + 1) / gridDim.x * p.subs;
  } else {
    blk_lo = p.nblk_full * (long long)blockIdx.x / gridDim.x;
    blk_hi = p.nblk_full * (long long)(blockIdx.x + 1) / gridDim.x;
  }
  const int has_tail = (p.tail && blockIdx.x == gridDim.x - 1) ? 1 : 0;
  const int n_iter = has_tail + (int)((blk_hi - blk_lo + p.subs - 1) / p.subs);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
      mbar_init(smem_u32(&bar_r32[s]), 1);
      mbar_init(smem_u32(&bar_conv[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_acc_full[b]), 1);
      mbar_init(smem_u32(&bar_acc_empty[b]), 4);     // one arrival per read-back warp
    }
    mbar_init_fence();
  }
  // row groups that are never loaded (gradient groups wholly past row 2m, the padding group
  // after the r rows, and with rconv the r groups themselves, of which the converter rewrites
  // rows 0..2 only) are zeroed once
  const int lgroups = (p.rows_used + 7) >> 3;                    // gradient row groups that get loaded
  for (int s = 0; s < p.stages; ++s) {
    for (int g = 0; g < ngroups; ++g) {
      const bool loaded = paired ? (g < 16 ? (g & 7) < lgroups : (!(g & 1) && !rconv))
                                 : (g < lgroups || (g == ggroups && !rconv));
      if (loaded) continue;
      uint8_t *z = smem_raw + (tiles - smem_u32(smem_raw)) + (size_t)s * stage_bytes + (size_t)g * group_bytes;
      for (uint32_t o = threadIdx.x * 16; o < group_bytes; o += kThreads * 16)
        *reinterpret_cast<uint4 *>(z + o) = make_uint4(0, 0, 0, 0);
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // visible to the MMA's smem reads
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_sh)), "r"(512u) : "memory");   // two accumulators of 256 columns
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_sh;
  cdg_grid_dep_wait();            // r (as its bf16 split) is written by the launch before this one
  const long long deadline = clock64() + kWaitCycles;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int it = 0; it < n_iter && ok; ++it) {
        const int s = it % p.stages;
        if (it >= p.stages) ok = mbar_wait(smem_u32(&bar_empty[s]), ((it / p.stages) - 1) & 1, deadline);
        if (!ok) break;
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t base = tiles + s * stage_bytes;
        const uint32_t rbase = base + (paired ? 16 : ggroups) * group_bytes;   // the r rows (first half)
        // rconv: fp32 r of the nb blocks of a (half) stage, rbox blocks per copy, instead of the r rows
        const int nb = paired ? hb : p.subs;
        const uint32_t r32 = tiles + r32_off + (uint32_t)(s * p.subs) * 256u;
        const uint32_t rg_tx = rconv ? 0u : 1u;                               // r row groups a copy fills
        const uint32_t rbar = smem_u32(&bar_r32[s]);
        // the small copies of r go first and complete a barrier of their own, so that the
        // converter works while the rows of the stage are still landing
        if (rconv) mbar_expect_tx(rbar, (uint32_t)(paired ? 2 * nb : nb) * 256u);
        if (has_tail && it == 0) {
          // ragged block: 8-row 2-D boxes into block slot 0 of every loaded row group
          const int col = (int)(p.nblk_full * kSubCols);   // 128-byte aligned
          if (rconv) {
            for (int q = 0; q < nb; q += p.rbox) tma_load_2d(r32 + q * 256u, &tm_r32, col + q * kSubCols, 0, rbar);
            if (paired)      // the other half: columns past the end, read as zeros
              for (int q = 0; q < nb; q += p.rbox)
                tma_load_2d(r32 + (uint32_t)(nb + q) * 256u, &tm_r32, (int)((p.nblk_full + 1 + q) * kSubCols), 0, rbar);
          }
          mbar_expect_tx(full, (uint32_t)(lgroups + rg_tx) * (1024u + (paired ? group_bytes : 0u)));
          for (int g = 0; g < lgroups; ++g) tma_load_2d(base + g * group_bytes, &tm_g2, col, g * 8, full);
          if (!rconv) tma_load_2d(rbase, &tm_r2, col, 0, full);
          if (paired) {
            // the other half of the pair: blocks past the end, which the copies fill with zeros
            const int past = (int)p.nblk_full;
            const uint32_t hbase = base + 8 * group_bytes;
            if (p.g4 > 0) tma_load_4d(hbase, &tm_g4, 0, 0, past, 0, full);
            for (int g = p.g4; g < lgroups; ++g) tma_load_3d(hbase + g * group_bytes, &tm_g3, 0, g * 8, past, full);
            if (!rconv) tma_load_3d(rbase + 2 * group_bytes, &tm_r3, 0, 0, past, full);
          }
        } else if (paired) {
          const long long first = blk_lo + (long long)(it - has_tail) * p.subs;
          if (rconv)
            for (int hf = 0; hf < 2; ++hf)
              for (int q = 0; q < nb; q += p.rbox)
                tma_load_2d(r32 + (uint32_t)(hf * nb + q) * 256u, &tm_r32, (int)(first + (long long)hf * hb + q) * kSubCols, 0, rbar);
          mbar_expect_tx(full, 2u * (uint32_t)(lgroups + rg_tx) * group_bytes);
          for (int hf = 0; hf < 2; ++hf) {
            const int blk = (int)(first + (long long)hf * hb);
            const uint32_t hbase = base + hf * 8 * group_bytes;
            if (p.g4 > 0) tma_load_4d(hbase, &tm_g4, 0, 0, blk, 0, full);
            for (int g = p.g4; g < lgroups; ++g) tma_load_3d(hbase + g * group_bytes, &tm_g3, 0, g * 8, blk, full);
            if (!rconv) tma_load_3d(rbase + hf * 2 * group_bytes, &tm_r3, 0, 0, blk, full);
          }
        } else {
          const long long first = blk_lo + (long long)(it - has_tail) * p.subs;
          if (rconv)
            for (int q = 0; q < nb; q += p.rbox)
              tma_load_2d(r32 + q * 256u, &tm_r32, (int)(first + q) * kSubCols, 0, rbar);
          mbar_expect_tx(full, (uint32_t)(lgroups + rg_tx) * group_bytes);
          if (p.g4 > 0) tma_load_4d(base, &tm_g4, 0, 0, (int)first, 0, full);
          for (int g = p.g4; g < lgroups; ++g) tma_load_3d(base + g * group_bytes, &tm_g3, 0, g * 8, (int)first, full);
          if (!rconv) tma_load_3d(rbase, &tm_r3, 0, 0, (int)first, full);
        }
        issued = it + 1;
      }
      if (!ok) {
        atomicOr(status, CDG_ST_TIMEOUT);
        // let the copies already issued land before the CTA gives up its shared memory
        for (int it = max(0, issued - p.stages); it < issued; ++it) {
          mbar_wait(smem_u32(&bar_full[it % p.stages]), (it / p.stages) & 1, clock64() + kWaitCycles);
          if (rconv) mbar_wait(smem_u32(&bar_r32[it % p.stages]), (it / p.stages) & 1, clock64() + kWaitCycles);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    // The whole warp runs the loop converged and one elected lane issues: operands of
    // tcgen05.mma computed under a lane test would have to be moved into uniform registers one
    // by one (84 cycles per MMA were measured that way), operands of converged code start there.
    // kind::f16, D = f32, A = B = bf16, both K-major, M = 128, N = ncols
    const uint32_t mma_n = paired ? (rconv ? 144u : 160u) : (uint32_t)p.ncols;
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((mma_n >> 3) << 17) | ((128u >> 4) << 24);
    // The fp32 accumulation inside the tensor core truncates; over hundreds of thousands of
    // columns that becomes a visible bias on sums of same-sign products.  So the sum is kept
    // in TMEM only for `drain` iterations (about 4096 columns), then handed to the read-back
    // warps, which add the chunks in fp32 registers with round-to-nearest, while the MMAs
    // continue into the other accumulator buffer.
    bool ok = true;
    int s = 0, c = 0, in_chunk = 0;          // stage, chunk number, position inside the chunk
    uint32_t full_parity = 0;
    for (int it = 0; it < n_iter; ++it) {
      const int buf = c & 1;
      const bool chunk_start = in_chunk == 0;
      if (chunk_start && c >= 2) ok = mbar_wait(smem_u32(&bar_acc_empty[buf]), ((c >> 1) - 1) & 1, deadline);
      if (ok) ok = mbar_wait(smem_u32(&bar_full[s]), full_parity, deadline);
      if (ok && rconv) ok = mbar_wait(smem_u32(&bar_conv[s]), full_parity, deadline);   // the r rows are in place
      ok = __all_sync(0xffffffffu, ok);      // the lanes leave together
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      int cnt = 1;
      if (!(has_tail && it == 0)) {
        const long long first = blk_lo + (long long)(it - has_tail) * p.subs;
        cnt = paired ? hb : (int)min((long long)p.subs, blk_hi - first);   // blocks past blk_hi belong to the next CTA
      }
      const uint32_t acc = tmem_acc + (uint32_t)buf * 256u;
      const uint32_t sbase = tiles + (uint32_t)s * stage_bytes;
      const bool chunk_end = (in_chunk == p.drain - 1) || (it == n_iter - 1);
      for (int q = 0; q < cnt; ++q) {
        const uint64_t desc = umma_desc(sbase + q * 1024u, group_bytes);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          // 16 bf16 = 32 bytes further along K inside the swizzle row
          const uint64_t dk = desc + (uint64_t)(k4 * 2);
          if (elect_one()) umma_bf16(acc, dk, dk, idesc, !(chunk_start && q == 0 && k4 == 0));
        }
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bar_empty[s]));  // stage reusable once these MMAs have read it
        if (chunk_end) umma_commit(smem_u32(&bar_acc_full[buf]));   // chunk complete
      }
      if (++in_chunk == p.drain) { in_chunk = 0; ++c; }
      if (++s == p.stages) { s = 0; full_parity ^= 1u; }
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
  } else if (warp == 6) {
    // ---------------- converter of r: fp32 piece -> three bf16 rows hi + mid + lo = r ----------------
    // Written in the layout a TMA copy would have produced: row t (paired, second block: 3 + t)
    // of the 8-row r group of block q, 16-byte chunk (c / 8) ^ row of its 128-byte row (the
    // 128-byte swizzle; the other rows stay zero).  Same
    // three roundings as everywhere else r is split, so the products come out bit for bit alike.
    if (rconv) {
      const int nb = paired ? hb : p.subs;
      uint8_t *smem_tiles = smem_raw + (tiles - smem_u32(smem_raw));
      bool ok = true;
      int s = 0;
      uint32_t parity = 0;
      for (int it = 0; it < n_iter; ++it) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_r32[s]), parity, deadline));
        if (!ok) break;
        for (int hf = 0; hf < (paired ? 2 : 1); ++hf) {
          const float *src = reinterpret_cast<const float *>(smem_tiles + r32_off + (size_t)(s * p.subs + hf * nb) * 256);
          uint8_t *rg = smem_tiles + (size_t)s * stage_bytes + (size_t)(paired ? 16 : ggroups) * group_bytes;
          const int r0 = 3 * hf;                     // paired: the second block's rows follow the first's
          for (int idx = lane * 8; idx < nb * kSubCols; idx += 256) {
            const int q = idx >> 6, chunk = (idx & 63) >> 3;
            const float4 f0 = *reinterpret_cast<const float4 *>(src + idx);
            const float4 f1 = *reinterpret_cast<const float4 *>(src + idx + 4);
            const float v[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
            uint32_t hi[4], mid[4], lo[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              __nv_bfloat16 h2[2], m2[2], l2[2];
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float x = v[2 * j + e];
                h2[e] = __float2bfloat16_rn(x);
                const float r1 = x - __bfloat162float(h2[e]);
                m2[e] = __float2bfloat16_rn(r1);
                l2[e] = __float2bfloat16_rn(r1 - __bfloat162float(m2[e]));
              }
              hi[j] = (uint32_t)__bfloat16_as_ushort(h2[0]) | ((uint32_t)__bfloat16_as_ushort(h2[1]) << 16);
              mid[j] = (uint32_t)__bfloat16_as_ushort(m2[0]) | ((uint32_t)__bfloat16_as_ushort(m2[1]) << 16);
              lo[j] = (uint32_t)__bfloat16_as_ushort(l2[0]) | ((uint32_t)__bfloat16_as_ushort(l2[1]) << 16);
            }
            uint8_t *blk = rg + (size_t)q * 1024;
            *reinterpret_cast<uint4 *>(blk + (r0 + 0) * 128 + ((chunk ^ (r0 + 0)) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4 *>(blk + (r0 + 1) * 128 + ((chunk ^ (r0 + 1)) << 4)) = make_uint4(mid[0], mid[1], mid[2], mid[3]);
            *reinterpret_cast<uint4 *>(blk + (r0 + 2) * 128 + ((chunk ^ (r0 + 2)) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMA reads these bytes through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_conv[s]));
        if (++s == p.stages) { s = 0; parity ^= 1u; }
      }
      if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
    }
  } else {
    // ---------------- accumulator read-back: TMEM chunks -> fp32 registers -> partial H ----------------
    const int lg = warp & 3;                 // TMEM lane group this warp may read
    const int row = lg * 32 + lane;
    const int nchunks = (n_iter + p.drain - 1) / p.drain;
    float accr[kMaxCols];
#pragma unroll
    for (int j = 0; j < kMaxCols; ++j) accr[j] = 0.f;
    bool ok = true;
    for (int c = 0; c < nchunks && ok; ++c) {
      const int buf = c & 1;
      ok = mbar_wait(smem_u32(&bar_acc_full[buf]), (c >> 1) & 1, deadline);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int piece = 0; piece < kMaxCols / 16; ++piece) {
        if (piece * 16 < p.ncols) {
          uint32_t v[16];
          // paired: rows 0..63 own D columns 0..63 and 128..143, rows 64..127 own 64..127 and 144..159
          // (rconv: both halves' b columns lie in piece 8, the upper rows' three at offset 3)
          const int src = paired ? (piece < 4 ? piece + 4 * (lg >> 1) : 8 + (rconv ? 0 : (lg >> 1))) : piece;
          const uint32_t taddr = tmem_acc + (uint32_t)buf * 256u + ((uint32_t)(lg * 32) << 16) + (uint32_t)(src * 16);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
              "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
                "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
                "=r"(v[14]), "=r"(v[15])
              : "r"(taddr) : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < 16; ++j) accr[piece * 16 + j] += __uint_as_float(v[j]);
        }
      }
      // the buffer may be overwritten once all four warps have read it
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
    }
    if (!ok && lane == 0) atomicOr(status, CDG_ST_TIMEOUT);
    if (paired) {
      // rows 64..127 hold the same entries of H for the other block of each pair: add them to
      // rows 0..63 through the (now idle) stage ring; only the four read-back warps take part
      float *xch = reinterpret_cast<float *>(smem_raw + (tiles - smem_u32(smem_raw)));
      if (lg >= 2) {
        if (rconv) {       // the upper rows' b columns sit three to the right of the lower rows'
#pragma unroll
          for (int j = 64; j < 67; ++j) accr[j] = accr[j + 3];
        }
#pragma unroll
        for (int j = 0; j < 80; ++j) xch[(row & 63) * 81 + j] = accr[j];
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (lg < 2) {
#pragma unroll
        for (int j = 0; j < 80; ++j) accr[j] += xch[row * 81 + j];
      }
    }
    if (row < p.rows_used && !(paired && lg >= 2)) {
      float *dst = partials + ((size_t)blockIdx.x * 128 + row) * (size_t)p.ncols;
#pragma unroll
      for (int piece = 0; piece < kMaxCols / 16; ++piece) {
        if (piece * 16 < p.ncols) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4 *>(dst + piece * 16 + j) =
                make_float4(accr[piece * 16 + j], accr[piece * 16 + j + 1], accr[piece * 16 + j + 2],
                            accr[piece * 16 + j + 3]);
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

// G and b from the per-CTA partial H in fp64.  A warp handles one entry (e < m*m: (k, i) =
// (e / m, e % m);  m*m <= e < m*m + m: b_i): lane l adds the CTAs l, l+32, ... in that order, the
// 32 lane sums are then added by a fixed butterfly.  Eight entries per block spread the loads
// over many SMs (an SM can keep only so many of these scattered loads in flight).
__global__ void __launch_bounds__(256)
umma_combine_kernel(const float *__restrict__ partials, int ctas, int ncols, int box_rows, int m,
                    double *__restrict__ gram, int *__restrict__ status, const CdgTail tail) {
  __shared__ double scan_sh[4 * 64 + 64 * 64];     // m <= 64 on this path
  __shared__ int is_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  cdg_grid_dep_wait();            // the partial H come from the launch before this one
  const int total = m * m + m;
  const int e = blockIdx.x * 8 + warp;
  const size_t cs = (size_t)128 * ncols;   // one CTA's partial H
  double acc = 0.0;
  if (e < m * m) {
    const int k = e / m, i = e % m;
    const size_t o00 = (size_t)k * ncols + i, o01 = o00 + m, o10 = (size_t)(m + k) * ncols + i, o11 = o10 + m;
#pragma unroll 5
    for (int c = lane; c < ctas; c += 32) {
      const float *P = partials + (size_t)c * cs;
      acc += ((double)P[o00] - (double)P[o01]) - ((double)P[o10] - (double)P[o11]);
    }
  } else if (e < total) {
    const int i = e - m * m;
    const size_t o0 = (size_t)i * ncols + box_rows, o1 = (size_t)(m + i) * ncols + box_rows;
#pragma unroll 5
    for (int c = lane; c < ctas; c += 32) {
      const float *P = partials + (size_t)c * cs;
      acc += (((double)P[o0] - (double)P[o1]) + ((double)P[o0 + 1] - (double)P[o1 + 1])) +
             ((double)P[o0 + 2] - (double)P[o1 + 2]);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0 && e < total) gram[e] = acc;
  if (!tail.enabled) return;

  // ---- the block that takes the last ticket has all of (G, b) before it: it decides ----
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(tail.ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const ScanSmem S = scan_smem(scan_sh, m);
  for (int j = threadIdx.x; j < m; j += blockDim.x) S.t[j] = __ldcg(gram + (size_t)m * m + j);
  for (int q = threadIdx.x; q < m * m; q += blockDim.x) S.g[q] = __ldcg(gram + q);
  scan_load_pairs(S, tail.perm_cur, m, tail.n, tail.k);
  if (threadIdx.x == 0) *tail.ticket = 0u;                    // ready for the next launch
  __syncthreads();
  scan_decide_and_write(S, S.g, m, tail.n, tail.k, tail.perm_next, tail.signs, tail.margins, tail.rnorm2, status,
                        tail.rule);
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
    else
      cudaGetLastError();
  }
  return fn;
}

// 2-D bf16 map over `rows` rows of `d` columns, row pitch `pitch_elems`, box [8 rows][64]
bool encode_map_2d(CUtensorMap *map, const void *base, long long d, int rows, long long pitch_elems) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
  cuuint32_t box[2] = {(cuuint32_t)kSubCols, 8};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view {64 columns, rows, nblk blocks of 64 columns} of the same memory (block pitch 128 bytes),
// box {64, 8 rows, subs blocks}
bool encode_map_3d(CUtensorMap *map, const void *base, long long nblk, int rows, long long pitch_elems, int subs) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)kSubCols, (cuuint64_t)rows, (cuuint64_t)nblk};
  cuuint64_t strides[2] = {(cuuint64_t)pitch_elems * 2, (cuuint64_t)kSubCols * 2};
  cuuint32_t box[3] = {(cuuint32_t)kSubCols, 8, (cuuint32_t)subs};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 4-D view {64 columns, 8 rows of a group, nblk blocks, groups} of the same memory; one box
// {64, 8, blocks, groups} lands as [group][block][8 rows][128 B], the layout the per-group boxes build
bool encode_map_4d(CUtensorMap *map, const void *base, long long nblk, int groups, long long pitch_elems, int blocks) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)kSubCols, 8, (cuuint64_t)nblk, (cuuint64_t)groups};
  cuuint64_t strides[3] = {(cuuint64_t)pitch_elems * 2, (cuuint64_t)kSubCols * 2, (cuuint64_t)pitch_elems * 16};
  cuuint32_t box[4] = {(cuuint32_t)kSubCols, 8, (cuuint32_t)blocks, (cuuint32_t)groups};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D fp32 map over r viewed as one row of d columns, box {blocks x 64 columns, 1 row}, no swizzle;
// columns past d read as zeros
bool encode_map_r32(CUtensorMap *map, const void *base, long long d, int blocks) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, 1};
  cuuint64_t strides[1] = {(cuuint64_t)d * 4};
  cuuint32_t box[2] = {(cuuint32_t)(blocks * kSubCols), 1};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Self-test of the bounded wait every TMA-fed kernel here relies on: one thread waits on a
// barrier that nothing ever completes, gives up after `cycles`, raises the time-out bit and
// returns.  No copy, no TMEM, nothing in flight.
__global__ void wait_timeout_selftest_kernel(long long cycles, int *status, long long *waited) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_init_fence();
    const long long t0 = clock64();
    const bool ok = mbar_wait(smem_u32(&bar), 0, t0 + cycles);
    *waited = clock64() - t0;
    if (!ok) atomicOr(status, CDG_ST_TIMEOUT);
  }
}

cudaError_t cdg_launch_wait_selftest(cdgrab_ctx *h, long long cycles, long long *waited_dev, cudaStream_t st) {
  wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(cycles, h->status, waited_dev);
  h->launches++;
  return cudaGetLastError();
}

void *cdg_tensor_map_encoder() { return (void *)encode_fn(); }

bool cdg_umma_supported(int m, long long d, int dtype) {
  // rows whose pitch is a multiple of 16 bytes
  if (dtype == CDGRAB_F32) {
    // fp32 gradients: the differences go in as three bf16 terms each, formed inside the kernel
    // (CDGRAB_UMMA_F32=0: fp32 gradients stay off the tensor cores)
    const char *e = getenv("CDGRAB_UMMA_F32");
    if (e && !strcmp(e, "0")) return false;
    return cdg_umma_f32_supported(m, d);
  }
  if (d % 8 != 0 || d < 4096 || encode_fn() == nullptr) return false;
  // bf16 gradients: the 2m rows fit one 128-row MMA tile
  return m <= 64;
}

int cdg_umma_setup(cdgrab_ctx *h) {
  if (h->dtype == CDGRAB_F32) return cdg_umma_f32_setup(h);
  h->umma_rows = 2 * h->m;
  h->umma_paired = (h->umma_rows <= 64) ? 1 : 0;  // CDGRAB_UMMA_PAIRED=0: one block per MMA
  if (const char *e = getenv("CDGRAB_UMMA_PAIRED")) {
    if (atoi(e) == 0) h->umma_paired = 0;
  }
  const int box_rows = h->umma_paired ? 64 : ((h->umma_rows + 15) / 16) * 16;
  h->umma_box_rows = box_rows;
  h->umma_ncols = box_rows + kRBoxRows;
  // 64-column blocks per stage: stages of roughly 70-80 KB measured best (4 blocks at m = 64,
  // 6-8 at m = 32); CDGRAB_UMMA_SUBS overrides
  int subs = 76 / (h->umma_ncols / 8);
  subs = subs < 2 ? 2 : (subs > 8 ? 8 : subs);
  if (h->umma_paired) subs = 6;                  // four stages of 54 KB (three of 60 KB with the r rows from HBM)
  if (const char *e = getenv("CDGRAB_UMMA_SUBS")) {
    const int v = atoi(e);
    if (v >= 1 && v <= (h->umma_paired ? 10 : 8)) subs = v;
  }
  if (h->umma_paired && (subs & 1)) ++subs;      // two halves per stage
  h->umma_subs_per_stage = subs;
  // TMEM chunk length in pipeline iterations (about 4096 columns); CDGRAB_UMMA_DRAIN overrides
  const int chunk_cols = 4096;
  h->umma_drain = chunk_cols / (subs * kSubCols) > 0 ? chunk_cols / (subs * kSubCols) : 1;
  if (const char *e = getenv("CDGRAB_UMMA_DRAIN")) {
    const int v = atoi(e);
    if (v >= 1 && v <= (1 << 20)) h->umma_drain = v;
  }
  // r reaches the MMA as three bf16 rows.  Default: pass 1 reads r itself (fp32, 4 bytes per
  // column) and one warp writes the rows in shared memory; CDGRAB_UMMA_RCONV=0: pass 2 keeps a
  // bf16 copy [3][d_pad] in HBM (6 bytes per column written, 6 read) and the TMA brings its rows.
  h->umma_rconv = 1;
  if (const char *e = getenv("CDGRAB_UMMA_RCONV")) h->umma_rconv = atoi(e) ? 1 : 0;
  {
    const int nb = h->umma_paired ? subs / 2 : subs;       // blocks per (half) stage
    int rbox = nb < 4 ? nb : 4;                            // at most 256 fp32 columns per copy
    while (nb % rbox) --rbox;
    h->umma_rbox = rbox;
  }
  const size_t group_bytes = (size_t)(h->umma_paired ? subs / 2 : subs) * 1024;
  // paired: 20 row groups per stage, 18 when the converter packs both blocks' r rows into one
  const int ngroups = h->umma_paired ? (h->umma_rconv ? 18 : 20) : h->umma_ncols / 8;
  const size_t stage_bytes = group_bytes * ngroups;
  const size_t slack = (ngroups < 16) ? (16 - ngroups) * group_bytes : 0;  // operand A spans 16 row groups
  const size_t r32_stage = h->umma_rconv ? (size_t)subs * 256 : 0;         // fp32 r of a stage
  const size_t budget = 226 * 1024 - 1024 - slack;
  int stages = (int)(budget / (stage_bytes + r32_stage));
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return CDGRAB_ERR_INVALID;
  h->umma_stages = stages;
  h->umma_smem = stages * (stage_bytes + r32_stage) + slack + 1024;
  const long long nblk_full = h->d / kSubCols;
  const long long total_sub = (h->d + kSubCols - 1) / kSubCols;
  h->umma_ctas = (int)((nblk_full < h->num_sms) ? (nblk_full > 0 ? nblk_full : 1) : h->num_sms);
  if (h->umma_paired) {
    const long long units = (nblk_full + subs - 1) / subs;
    h->umma_ctas = (int)(units < h->num_sms ? (units > 0 ? units : 1) : h->num_sms);
  }
  h->d_pad = total_sub * kSubCols;
  if (cdg_alloc(h, &h->umma_partials, sizeof(float) * 128 * (size_t)h->umma_ncols * h->umma_ctas) != cudaSuccess ||
      (!h->umma_rconv && cdg_alloc(h, &h->r_split, sizeof(__nv_bfloat16) * 3 * (size_t)h->d_pad) != cudaSuccess)) {
    cudaGetLastError();
    return CDGRAB_ERR_NOMEM;
  }
  if (cudaMemset(h->umma_partials, 0, sizeof(float) * 128 * (size_t)h->umma_ncols * h->umma_ctas) != cudaSuccess)
    return CDGRAB_ERR_CUDA;
  if (h->umma_rconv) {
    if (!encode_map_r32(&h->tm_r32, h->r, h->d, h->umma_rbox)) return CDGRAB_ERR_CUDA;
    h->tm_r = h->tm_r32;               // unused by the kernel in this mode; any valid map will do
    h->tm_r2 = h->tm_r32;
  } else {
    if (cudaMemset(h->r_split, 0, sizeof(__nv_bfloat16) * 3 * (size_t)h->d_pad) != cudaSuccess) return CDGRAB_ERR_CUDA;
    if (!encode_map_3d(&h->tm_r, h->r_split, nblk_full, 3, h->d_pad, h->umma_paired ? subs / 2 : subs))
      return CDGRAB_ERR_CUDA;
    if (!encode_map_2d(&h->tm_r2, h->r_split, h->d, 3, h->d_pad)) return CDGRAB_ERR_CUDA;
    h->tm_r32 = h->tm_r;               // unused by the kernel in this mode
  }
  if (cdg_open_smem_limit(gram_umma_kernel) !=
      cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  // one copy for all full row groups of a (half) stage; CDGRAB_UMMA_G4=0: per-group copies only
  h->umma_g4 = h->umma_rows / 8;
  if (const char *e = getenv("CDGRAB_UMMA_G4")) {
    if (atoi(e) == 0) h->umma_g4 = 0;
  }
  if (h->d * 16 >= (1ll << 40)) h->umma_g4 = 0;             // the group stride must fit the map
  h->umma_fused = h->shard ? 0 : 1;      // a shard's decisions wait for the sum over shards
  if (const char *e = getenv("CDGRAB_UMMA_FUSE_TAIL")) {
    if (atoi(e) == 0) h->umma_fused = 0;
  }
  return CDGRAB_OK;
}

void cdg_umma_teardown(cdgrab_ctx *h) {
  cdg_umma_f32_teardown(h);
  cdg_free(h->r_split);
  cdg_free(h->umma_partials);
  h->r_split = nullptr;
  h->umma_partials = nullptr;
}

cudaError_t cdg_launch_gram_umma(cdgrab_ctx *h, const void *grads, cudaStream_t st) {
  if (h->umma_f32) return cdg_launch_gram_umma_f32(h, grads, st);
  const long long nblk_full = h->d / kSubCols;
  const void *src = grads;             // the MMA's rows are the caller's bf16 gradients as they lie in HBM
  const long long pitch = h->d;
  const int rows = h->umma_rows;
  int slot = h->tm_g.find(src);
  if (slot < 0) {
    slot = h->tm_g.victim();
    CUtensorMap *mp = h->tm_g.maps[slot];
    const int box_blocks = h->umma_paired ? h->umma_subs_per_stage / 2 : h->umma_subs_per_stage;
    if (!encode_map_3d(&mp[0], src, nblk_full, rows, pitch, box_blocks) || !encode_map_2d(&mp[1], src, h->d, rows, pitch))
      return cudaErrorInvalidValue;
    // a driver that refuses the 4-D map sends this handle to per-group copies for good
    if (h->umma_g4 > 0 && !encode_map_4d(&mp[2], src, nblk_full, h->umma_g4, pitch, box_blocks)) h->umma_g4 = 0;
    if (h->umma_g4 == 0) mp[2] = mp[0];
    h->tm_g.commit(slot, src);
  }
  const CUtensorMap *mp = h->tm_g.maps[slot];
  UmmaParams p;
  p.box_rows = h->umma_box_rows;
  p.ncols = h->umma_ncols;
  p.rows_used = rows;
  p.subs = h->umma_subs_per_stage;
  p.stages = h->umma_stages;
  p.nblk_full = nblk_full;
  p.tail = (h->d % kSubCols) ? 1 : 0;
  p.drain = h->umma_drain;
  p.g4 = h->umma_g4;
  p.paired = h->umma_paired;
  p.rconv = h->umma_rconv;
  p.rbox = h->umma_rbox;
  {
    CdgProfScope ps(h, CDGRAB_K_GRAM, st);
    cdg_launch_dep(h, gram_umma_kernel, dim3(h->umma_ctas), dim3(kThreads), h->umma_smem, st, mp[0], h->tm_r,
                   mp[1], h->tm_r2, mp[2], h->tm_r32, p, h->umma_partials, h->status);
  }
  {
    CdgProfScope ps(h, CDGRAB_K_COMBINE, st);
    const int total = h->m * h->m + h->m;
    cdg_launch_dep(h, umma_combine_kernel, dim3((total + 7) / 8), dim3(256), 0, st, h->umma_partials, h->umma_ctas,
                   h->umma_ncols, h->umma_box_rows, h->m, h->gram, h->status,
                   cdg_tail_of(h, h->umma_fused));
  }
  return cudaGetLastError();
}
