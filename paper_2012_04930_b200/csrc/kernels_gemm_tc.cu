// C = epi(A B^T) on the 5th-generation tensor cores with fp32-level accuracy:
// the dense feature transform H W and the gradient products of the GCN layer
// (Section 4.1) as tcgen05.mma kind::tf32 with a three-term operand split.
//
// Every fp32 operand x is split into hi = x with the low 13 mantissa bits cleared
// (exactly a TF32 number; the tensor core takes it from the raw fp32 word, whose
// low bits it does not read) and lo = x - hi (exact in fp32, itself cut to TF32
// by the tensor core).  A B^T ~= A_hi B_hi^T + A_lo B_hi^T + A_hi B_lo^T; the dropped
// term and the rounding of lo are O(2^-21) relative, well inside the 1e-4 bar
// that plain TF32 (2^-11 per operand) misses.
//
// One CTA computes one 128 x BN tile (optionally one k-slice of it).  Warp 0
// streams fp32 boxes of both operands into shared memory with TMA (128-byte
// swizzle): an operand whose K index is contiguous in memory arrives K-major
// (one 32 x rows box), one whose M / N index is contiguous arrives MN-major
// (32 x 32 boxes, one per 32 rows), so neither H W nor H^T Q needs a
// transposed copy.  Warps 2-9 write the lo part of every stage into a second
// buffer (a K-major A operand: hi and lo part into tensor memory), warp 1 issues the MMAs - A_hi [B_hi | B_lo] as one instruction of
// twice the tile's columns, then A_lo B_hi - into two TMEM accumulators, and
// warps 2-9 finally read the accumulators back, add them, turn the sum through shared memory
// so that global accesses are row-contiguous, and apply the epilogue.  All
// waits are bounded (tens of milliseconds; a healthy phase takes microseconds):
// a wait that runs out sets an error word that the host reads
// (gcnsa_tc_status) and the CTA winds down.  The word is sticky: waiting threads
// poll it and give up at once when another CTA has set it, and a launch that
// finds it set returns before it allocates anything, until gcnsa_tc_clear.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "internal.h"

namespace gcnsa {

namespace {

constexpr int BM = 128, BK = 32;
constexpr int kSplitWarps = 8;
constexpr int kThreads = 64 + 32 * kSplitWarps;
constexpr int A_BYTES = BM * BK * 4;             // 16 KiB
constexpr long long kSpinCycles = 100000000LL;  // about 50 ms; a healthy wait ends within microseconds
constexpr long long kPollCycles = 1LL << 16;    // a waiting thread looks at the error word this often (~33 us)

__device__ int g_tc_error = 0;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ int tc_error_now() { return *reinterpret_cast<volatile int*>(&g_tc_error); }

// Bounded wait: false when the phase did not complete within kSpinCycles, or when the error word has been set in
// the meantime (by this CTA, another one, or an earlier launch).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  long long t_poll = t0;
  while (!mbar_try_wait(bar, parity)) {
    const long long now = clock64();
    if (now - t_poll > kPollCycles) {
      if (tc_error_now() != 0) return false;
      t_poll = now;
    }
    if (now - t0 > kSpinCycles) {
      atomicCAS(&g_tc_error, 0, code);
      return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// K-major operand tile in shared memory, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);  // start address
  d |= (uint64_t)1 << 16;                       // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                       // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                       // SWIZZLE_128B
  return d;
}

// MN-major operand tile of 32-bit elements: the 128-byte swizzle with 32-byte atoms is the one layout the tensor
// core transposes.  Blocks of 32 rows (M or N) x 32 k; inside a block the 32 elements of one k are contiguous
// (128 bytes), 4 k form a 512-byte swizzle group, blocks are 4096 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(4096 >> 4) << 16;  // leading byte offset: next block of 32 rows
  d |= (uint64_t)(512 >> 4) << 32;   // stride byte offset: next group of 4 k
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)1 << 61;            // SWIZZLE_128B_BASE32B
  return d;
}

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// the same with the A operand in tensor memory (128 lanes = rows, one 32-bit column per k)
__device__ __forceinline__ void umma_tf32_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(tmem_d),
      "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// 16 consecutive columns of this thread's TMEM lane (lane quarter of the warp + lane id)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float epi_apply(float v, int epi, const float* __restrict__ aux, int64_t ldaux, int64_t i,
                                           int64_t j) {
  if (epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_BIAS_RELU) {
    if (aux) v += __ldg(aux + j);
    if (epi == GCNSA_EPI_BIAS_RELU) v = fmaxf(v, 0.f);
  } else if (epi == GCNSA_EPI_ROWSCALE) {
    v *= __ldg(aux + i);
  } else if (epi == GCNSA_EPI_MASK) {
    v = __ldg(aux + i * ldaux + j) > 0.f ? v : 0.f;
  }
  return v;
}

// lo = x - hi with hi = x with its 13 low mantissa bits cleared (second buffer, same offsets).  The first buffer
// keeps the raw fp32 words: kind::tf32 reads the sign, exponent and upper 10 mantissa bits of each word, which is
// exactly hi, so rewriting it would only cost shared-memory bandwidth, the unit this loop is bound by (per k-block:
// 32 KB landed by TMA, 32 KB read and 32 KB written here, 96 KB read by the twelve MMAs).  Measured: results equal
// with and without the masking store; the parity tests of the tensor-core path (2e-5 of max) would fail on a part
// that rounded instead (2^-12 per operand).
__device__ __forceinline__ void split_buffer(const uint8_t* hi_buf, uint8_t* lo_buf, int bytes, int t) {
#pragma unroll 4
  for (int i = t; i < bytes / 16; i += 32 * kSplitWarps) {
    const uint4* hp = reinterpret_cast<const uint4*>(hi_buf) + i;
    const uint4 x = *hp;
    uint4 h;
    h.x = x.x & 0xFFFFE000u; h.y = x.y & 0xFFFFE000u; h.z = x.z & 0xFFFFE000u; h.w = x.w & 0xFFFFE000u;
    float4 l;
    l.x = __uint_as_float(x.x) - __uint_as_float(h.x);
    l.y = __uint_as_float(x.y) - __uint_as_float(h.y);
    l.z = __uint_as_float(x.z) - __uint_as_float(h.z);
    l.w = __uint_as_float(x.w) - __uint_as_float(h.w);
    reinterpret_cast<float4*>(lo_buf)[i] = l;
  }
}

// STAGES: 3 (one CTA per SM), or 2 for 64-column tiles, whose 48 KiB stages then let two CTAs share an SM: products
// with a short inner dimension are dominated by the fixed latency of a CTA (first loads, accumulator turn, stores),
// which a second resident CTA overlaps.
template <int BN, bool A_MN, bool B_MN, int STAGES>
__global__ void __launch_bounds__(kThreads, (STAGES == 2 ? 2 : 1))
gemm_tf32x3(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int64_t M, int64_t N,
            int k_blocks, int k_blocks_per_split, float* __restrict__ c, int64_t ldc, int accumulate, int epi,
            const float* __restrict__ aux, int64_t ldaux, float* __restrict__ partial, int vec_ok, int terms) {
  constexpr int B_BYTES = BN * BK * 4;
  constexpr int STAGE_BYTES = 2 * A_BYTES + 2 * B_BYTES;
  // The hi and lo tiles of B lie next to each other in a stage, so A_hi [B_hi | B_lo] is ONE instruction of 2 BN
  // columns into two accumulators (columns [0, BN) and [BN, 2 BN) of TMEM) that the epilogue adds; with A_lo B_hi that
  // makes two instructions per 8 k instead of three.  Measured with clock64 around the issue loop: a k-block of
  // 128 x 128 x 32 then takes the issuing thread about 800 clocks, which is the TF32 rate of the tensor pipe for
  // the 3 x 128 x 128 x 32 products (about 2000 multiply-adds per clock and SM); three separate instructions took 1000.
  constexpr int ACC_COLS = 2 * BN;
  static_assert(ACC_COLS <= 256, "one instruction covers at most 256 columns");
  // A K-major operand does not go back to shared memory after the split: the split warps, which hold its values in
  // registers anyway, store the hi and the lo part into tensor memory (one lane per row, 32 + 32 columns per stage)
  // and the MMAs read A from there.  Shared memory then carries 128 instead of 176 KiB per 128 x 128 x 32 k-block:
  // no A_lo tile is written and the MMAs read no A tile.  Measured gain: 1 to 2 % of the products' time.
  constexpr bool A_TMEM = !A_MN;
  constexpr int A_COLS = A_TMEM ? STAGES * 64 : 0;
  constexpr int TMEM_COLS = (ACC_COLS + A_COLS) <= 128 ? 128 : ((ACC_COLS + A_COLS) <= 256 ? 256 : 512);
  static_assert(ACC_COLS + A_COLS <= 512, "tensor memory has 512 columns");
  // two CTAs share an SM only in the two-stage variant: both must fit the 512 columns
  static_assert(STAGES != 2 || TMEM_COLS <= 256, "two resident CTAs");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* full = bars;                // TMA landed                 (1 arrival + bytes)
  uint64_t* split = bars + STAGES;      // hi / lo written            (one arrival per split warp)
  uint64_t* empty = bars + 2 * STAGES;  // MMAs of the stage retired  (1 arrival by tcgen05.commit)
  uint64_t* accum = bars + 3 * STAGES;  // accumulator complete
  uint64_t* drain = bars + 3 * STAGES + 1;  // wind-down only: the MMAs issued before a failed wait have retired
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * STAGES + 2);
  int* abort_slot = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const int kb0 = blockIdx.z * k_blocks_per_split;
  const int kb1 = min(k_blocks, kb0 + k_blocks_per_split);
  const int n_kb = max(kb1 - kb0, 0);

  // a wait ran out in an earlier launch or in another CTA of this one: nothing is allocated, nothing is computed
  if (threadIdx.x == 0) *abort_slot = tc_error_now();
  __syncthreads();
  if (*abort_slot != 0) return;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&split[s], kSplitWarps);
      mbar_init(&empty[s], 1);
    }
    mbar_init(accum, 1);
    mbar_init(drain, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        ok = mbar_wait(&empty[s], ph ^ 1, 1);
        if (!ok) break;
        uint8_t* st = smem + s * STAGE_BYTES;
        mbar_expect_tx(&full[s], A_BYTES + B_BYTES);
        const int kx = (kb0 + it) * BK;
        if (A_MN) {
#pragma unroll
          for (int j = 0; j < BM / 32; ++j) tma_load_2d(st + j * 4096, &map_a, (int)m0 + 32 * j, kx, &full[s]);
        } else {
          tma_load_2d(st, &map_a, kx, (int)m0, &full[s]);
        }
        if (B_MN) {
#pragma unroll
          for (int j = 0; j < BN / 32; ++j)
            tma_load_2d(st + 2 * A_BYTES + j * 4096, &map_b, (int)n0 + 32 * j, kx, &full[s]);
        } else {
          tma_load_2d(st + 2 * A_BYTES, &map_b, kx, (int)n0, &full[s]);
        }
        issued = it + 1;
      }
      if (!ok || tc_error_now() != 0) {  // wind down: let the copies already issued land before the CTA exits
        const long long t0 = clock64();
        for (int it = max(issued - STAGES, 0); it < issued; ++it) {
          uint64_t* b = &full[it % STAGES];
          const uint32_t ph = (it / STAGES) & 1;
          while (!mbar_try_wait(b, ph) && clock64() - t0 < kSpinCycles) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B tf32, both K-major, N x 128
      const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      const uint32_t idesc2 = (idesc & ~(0x3Fu << 17)) | ((uint32_t)((2 * BN) >> 3) << 17);  // the same with 2 BN columns
      bool ok = true;
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        ok = mbar_wait(&split[s], ph, 3);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t base = smem_u32(smem + s * STAGE_BYTES);
        const uint64_t a_hi = A_MN ? umma_desc_mn(base) : umma_desc(base);
        const uint64_t a_lo = A_MN ? umma_desc_mn(base + A_BYTES) : umma_desc(base + A_BYTES);
        const uint64_t b_hi = B_MN ? umma_desc_mn(base + 2 * A_BYTES) : umma_desc(base + 2 * A_BYTES);
        const uint64_t b_lo = B_MN ? umma_desc_mn(base + 2 * A_BYTES + B_BYTES) : umma_desc(base + 2 * A_BYTES + B_BYTES);
#pragma unroll
        for (int k = 0; k < BK / 8; ++k) {
          // one MMA covers 8 k: 32 bytes further inside the swizzle atom (K-major) or the next 1024-byte group (MN-major)
          const uint64_t adv_a = (uint64_t)((A_MN ? k * 1024 : k * 32) >> 4);
          const uint64_t adv_b = (uint64_t)((B_MN ? k * 1024 : k * 32) >> 4);
          if (terms == 3) {
            if constexpr (A_TMEM) {
              const uint32_t ta = tmem_base + (uint32_t)(ACC_COLS + s * 64 + 8 * k);
              umma_tf32_ta(tmem_base, ta, b_hi + adv_b, idesc2, (it | k) != 0);       // A_hi [B_hi | B_lo]
              umma_tf32_ta(tmem_base, ta + 32, b_hi + adv_b, idesc, 1);               // + A_lo B_hi on the first half
            } else {
              umma_tf32(tmem_base, a_hi + adv_a, b_hi + adv_b, idesc2, (it | k) != 0);
              umma_tf32(tmem_base, a_lo + adv_a, b_hi + adv_b, idesc, 1);
            }
          } else if constexpr (A_TMEM) {  // plain TF32: the leading parts only
            umma_tf32_ta(tmem_base, tmem_base + (uint32_t)(ACC_COLS + s * 64 + 8 * k), b_hi + adv_b, idesc, (it | k) != 0);
          } else {
            umma_tf32(tmem_base, a_hi + adv_a, b_hi + adv_b, idesc, (it | k) != 0);
          }
        }
        umma_commit(&empty[s]);  // arrives when the MMAs above have finished reading this stage
      }
      if (ok && n_kb > 0) {
        umma_commit(accum);
      } else if (n_kb > 0) {
        // a wait ran out: the MMAs issued so far must have retired before the accumulator columns are given back
        umma_commit(drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(drain, 0) && clock64() - t0 < kSpinCycles) {
        }
      }
    }
  } else {
    // ---------------- operand split, then epilogue (warps 2..9) ----------------
    const int t = threadIdx.x - 64;
    bool ok = true;
    for (int it = 0; it < n_kb; ++it) {
      const int s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1;
      ok = mbar_wait(&full[s], ph, 4);
      if (!ok) break;
      uint8_t* st = smem + s * STAGE_BYTES;
      if constexpr (A_TMEM) {
        // thread = row 32 q + lane of the A tile (q = the lane quarter of tensor memory this warp may touch), the two
        // warps of a quarter take 16 k each: four 16-byte chunks of the row (128-byte swizzle: chunk c of row r sits
        // at chunk position c ^ (r % 8)), both parts straight into tensor memory
        const int q = warp & 3, kh = (warp - 2) >> 2, row = 32 * q + lane;
        const uint8_t* arow = st + (row >> 3) * 1024 + (row & 7) * 128;
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const uint4 x = *reinterpret_cast<const uint4*>(arow + (((4 * kh + cc) ^ (row & 7)) << 4));
          hi[4 * cc + 0] = x.x; hi[4 * cc + 1] = x.y; hi[4 * cc + 2] = x.z; hi[4 * cc + 3] = x.w;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j)
          lo[j] = __float_as_uint(__uint_as_float(hi[j]) - __uint_as_float(hi[j] & 0xFFFFE000u));
        const uint32_t ta = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(ACC_COLS + s * 64 + 16 * kh);
        tmem_st16(ta, hi);  // the raw words: the tensor core reads their leading 19 bits
        if (terms == 3) tmem_st16(ta + 32, lo);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        if (terms == 3) split_buffer(st + 2 * A_BYTES, st + 2 * A_BYTES + B_BYTES, B_BYTES, t);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      } else if (terms == 3) {
        // elementwise, so the swizzled position of an element is the same in the hi and the lo buffer
        split_buffer(st, st + A_BYTES, A_BYTES, t);
        split_buffer(st + 2 * A_BYTES, st + 2 * A_BYTES + B_BYTES, B_BYTES, t);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA
      __syncwarp();
      if (lane == 0) mbar_arrive(&split[s]);
    }
    const int quad = warp & 3;         // the TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;  // warps 2-5: left half of the columns, 6-9: right half
    constexpr int CW = BN / 2;         // columns per warp
    constexpr int P = CW + 4;          // tile pitch in floats: 16-byte stores of 8 rows hit 8 different bank groups
    constexpr int LPR = CW / 4;        // lanes per row when every lane moves one float4
    constexpr int RPI = 32 / LPR;      // rows per warp instruction
    constexpr int NIT = 32 / RPI;      // float4 a thread stores
    // thread = (row within RPI, float4 column): row-contiguous global accesses, RPI rows per instruction
    const int lr = lane / LPR, lc = (lane % LPR) * 4;
    const int64_t col = n0 + half * CW + lc;
    const int64_t row_base = m0 + quad * 32;
    const bool vec_path = vec_ok && !partial && col + 3 < N;
    // the ReLU mask of this thread's part of the tile is fetched while the last MMAs run: all its loads are in
    // flight together instead of one per stored row segment after the accumulator is complete
    float4 mk[NIT];
    const bool masked = vec_path && epi == GCNSA_EPI_MASK;
    if (ok && masked) {
#pragma unroll
      for (int i = 0; i < NIT; ++i) {
        const int64_t row = row_base + lr + i * RPI;
        mk[i] = row < M ? __ldg(reinterpret_cast<const float4*>(aux + row * ldaux + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (ok && n_kb > 0) ok = mbar_wait(accum, 0, 5);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // every stage buffer is idle by now: 32 x P floats of it per warp turn the accumulator around
      float* tile = reinterpret_cast<float*>(smem) + (warp - 2) * (32 * P);
      // a row scale is applied here, where a thread holds one row of the accumulator: one load per thread and tile
      const bool scale_here = epi == GCNSA_EPI_ROWSCALE && !partial;
      float row_scale = 1.f;
      if (scale_here) {
        const int64_t my_row = m0 + quad * 32 + lane;
        row_scale = my_row < M ? __ldg(aux + my_row) : 0.f;
        epi = GCNSA_EPI_NONE;
      }
#pragma unroll
      for (int c0 = 0; c0 < CW; c0 += 32) {
        uint32_t v[32];
        if (n_kb > 0) {
          tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * CW + c0), v);
          if (terms == 3) {  // the second accumulator: A_hi B_lo
            uint32_t u[32];
            tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(BN + half * CW + c0), u);
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(u[j]));
          }
          if (scale_here) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * row_scale);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 32; j += 4)  // thread = row
          *reinterpret_cast<uint4*>(tile + lane * P + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      }
      __syncwarp();
      const int64_t n_pad = min(ldc, (N + 3) / 4 * 4);
      if (vec_path) {
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
          const int r = lr + i * RPI;
          const int64_t row = row_base + r;
          if (row < M) {
            float4 a4 = *reinterpret_cast<const float4*>(tile + r * P + lc);
            float* dst = c + row * ldc + col;
            if (masked) {
              a4.x = mk[i].x > 0.f ? a4.x : 0.f; a4.y = mk[i].y > 0.f ? a4.y : 0.f;
              a4.z = mk[i].z > 0.f ? a4.z : 0.f; a4.w = mk[i].w > 0.f ? a4.w : 0.f;
            } else if (epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_BIAS_RELU) {
              if (aux) {
                const float4 b4 = __ldg(reinterpret_cast<const float4*>(aux + col));
                a4.x += b4.x; a4.y += b4.y; a4.z += b4.z; a4.w += b4.w;
              }
              if (epi == GCNSA_EPI_BIAS_RELU) {
                a4.x = fmaxf(a4.x, 0.f); a4.y = fmaxf(a4.y, 0.f); a4.z = fmaxf(a4.z, 0.f); a4.w = fmaxf(a4.w, 0.f);
              }
            }
            if (accumulate) {
              const float4 o = *reinterpret_cast<const float4*>(dst);
              a4.x += o.x; a4.y += o.y; a4.z += o.z; a4.w += o.w;
            }
            *reinterpret_cast<float4*>(dst) = a4;
          }
        }
      } else {
        for (int r = lr; r < 32; r += RPI) {
          const int64_t row = row_base + r;
          if (row >= M) break;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int64_t cc = col + e;
            const float acc = tile[r * P + lc + e];
            if (partial) {
              if (cc < N) partial[((int64_t)blockIdx.z * M + row) * N + cc] = acc;
            } else if (cc < N) {
              const float o = epi_apply(acc, epi, aux, ldaux, row, cc);
              float* dst = c + row * ldc + cc;
              *dst = accumulate ? *dst + o : o;
            } else if (cc < n_pad && !accumulate) {
              c[row * ldc + cc] = 0.f;
            }
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

// fp32 matrix with `inner` contiguous elements per line and `outer` lines, pitch ld floats; box = 32 x box_outer,
// 128-byte swizzle, zero fill outside.  K-major operand: inner = k, outer = rows, box_outer = tile rows.
// MN-major operand: inner = rows (M or N), outer = k, box_outer = 32, swizzle with 32-byte atoms.
bool make_map(CUtensorMap* map, const float* base, int64_t outer, int64_t inner, int64_t ld, int box_outer,
              bool mn_major) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
         CUDA_SUCCESS;
}

struct TcPlan {
  int bn, splits, k_blocks, kb_per_split;
  size_t partial_bytes;
};

TcPlan tc_plan(int64_t m, int64_t n, int64_t k) {
  TcPlan p;
  p.k_blocks = (int)((k + BK - 1) / BK);
  // 64-column tiles for narrow results and for an inner dimension of at most two k-blocks (the A tile re-read per
  // column tile is then small, and two CTAs per SM hide the fixed latency that dominates such products)
  p.bn = (n <= 64 || p.k_blocks <= 2) ? 64 : 128;
  const int64_t tiles = ((m + BM - 1) / BM) * ((n + p.bn - 1) / p.bn);
  int64_t splits = 1;
  // one CTA per SM: the k-slices of all tiles together must fit the 148 SMs in one wave (5 tiles x 30 slices would
  // leave two CTAs for a second wave that takes as long as the first)
  if (tiles < 74 && p.k_blocks >= 16) splits = std::min<int64_t>(148 / tiles, p.k_blocks / 8);
  splits = std::max<int64_t>(splits, 1);
  p.kb_per_split = (int)((p.k_blocks + splits - 1) / splits);
  p.splits = (p.k_blocks + p.kb_per_split - 1) / p.kb_per_split;
  if (p.splits < 1) p.splits = 1;
  auto up = [](size_t b) { return (b + 255) / 256 * 256; };
  p.partial_bytes = up(p.splits > 1 ? (size_t)p.splits * m * n * sizeof(float) : 0);
  return p;
}

template <int BN, bool A_MN, bool B_MN, int STAGES>
cudaError_t run_tc_stages(cudaStream_t s, const TcPlan& p, const CUtensorMap& ma, const CUtensorMap& mb, int64_t m,
                          int64_t n, float* c, int64_t ldc, int accumulate, int epi, const float* aux, int64_t ldaux,
                          float* partial, int vec_ok, int terms) {
  constexpr int smem = STAGES * (2 * A_BYTES + 2 * BN * BK * 4) + 1024 + 256;
  cudaError_t e0 =
      cudaFuncSetAttribute(gemm_tf32x3<BN, A_MN, B_MN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e0 != cudaSuccess) return e0;
  dim3 grid((unsigned)((n + BN - 1) / BN), (unsigned)((m + BM - 1) / BM), (unsigned)p.splits);
  gemm_tf32x3<BN, A_MN, B_MN, STAGES><<<grid, kThreads, smem, s>>>(ma, mb, m, n, p.k_blocks, p.kb_per_split, c, ldc,
                                                                   accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  note_launch();
  return cudaGetLastError();
}

template <int BN, bool A_MN, bool B_MN>
cudaError_t run_tc(cudaStream_t s, const TcPlan& p, const CUtensorMap& ma, const CUtensorMap& mb, int64_t m, int64_t n,
                   float* c, int64_t ldc, int accumulate, int epi, const float* aux, int64_t ldaux, float* partial,
                   int vec_ok, int terms) {
  if constexpr (BN == 64) {
    // more CTAs than SMs: two per SM with two stages each; a grid of one wave keeps the deeper pipeline
    const int64_t ctas = ((n + BN - 1) / BN) * ((m + BM - 1) / BM) * p.splits;
    if (ctas > 148)
      return run_tc_stages<BN, A_MN, B_MN, 2>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  }
  return run_tc_stages<BN, A_MN, B_MN, 3>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
}

template <int BN>
cudaError_t run_tc_major(bool a_mn, bool b_mn, cudaStream_t s, const TcPlan& p, const CUtensorMap& ma,
                         const CUtensorMap& mb, int64_t m, int64_t n, float* c, int64_t ldc, int accumulate, int epi,
                         const float* aux, int64_t ldaux, float* partial, int vec_ok, int terms) {
  if (a_mn && b_mn) return run_tc<BN, true, true>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  if (a_mn) return run_tc<BN, true, false>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  if (b_mn) return run_tc<BN, false, true>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  return run_tc<BN, false, false>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
}

}  // namespace

size_t gemm_tc_workspace(int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k) {
  (void)ta; (void)tb;  // operands are read in the layout they have: no transposed copies to make room for
  return tc_plan(m, n, k).partial_bytes;
}

// Returns 0 on success, a cudaError_t on a CUDA failure, -1 when this shape / alignment / workspace cannot take
// the tensor-core path (the caller then uses the fp32 FMA kernel).
int launch_gemm_tc(void* stream, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a, int64_t lda,
                   const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi, const float* aux,
                   int64_t ldaux, void* workspace, size_t workspace_bytes, int terms) {
  if (m <= 0 || n <= 0 || k <= 0 || m >= (1LL << 31) || n >= (1LL << 31) || k >= (1LL << 31)) return -1;
  cudaStream_t s = (cudaStream_t)stream;
  const TcPlan p = tc_plan(m, n, k);
  const size_t need = p.partial_bytes;
  if (need > workspace_bytes) return -1;
  if (need && (!workspace || ((uintptr_t)workspace & 255))) return -1;
  // TMA needs 16-byte aligned bases and pitches
  if (((uintptr_t)a & 15) || (lda % 4) || ((uintptr_t)b & 15) || (ldb % 4)) return -1;
  if (!encode_fn()) return -1;
  uint8_t* ws = (uint8_t*)workspace;
  float* partial = p.splits > 1 ? (float*)ws : nullptr;
  const bool a_mn = ta != 0;   // stored K x M: the M index is contiguous
  const bool b_mn = tb == 0;   // stored K x N: the N index is contiguous
  CUtensorMap ma, mb;
  const bool ok_a = a_mn ? make_map(&ma, a, k, m, lda, 32, true) : make_map(&ma, a, m, k, lda, BM, false);
  const bool ok_b = b_mn ? make_map(&mb, b, k, n, ldb, 32, true) : make_map(&mb, b, n, k, ldb, p.bn, false);
  if (!ok_a || !ok_b) return (int)cudaErrorInvalidValue;
  // float4 epilogue: C (and a mask) 16-byte aligned with pitches that are multiples of 4; a bias only needs alignment
  int vec_ok = (((uintptr_t)c & 15) == 0) && (ldc % 4 == 0);
  if (epi == GCNSA_EPI_MASK) vec_ok = vec_ok && (((uintptr_t)aux & 15) == 0) && (ldaux % 4 == 0);
  if ((epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_BIAS_RELU) && aux) vec_ok = vec_ok && (((uintptr_t)aux & 15) == 0);
  cudaError_t e = p.bn == 64
                      ? run_tc_major<64>(a_mn, b_mn, s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms)
                      : run_tc_major<128>(a_mn, b_mn, s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, partial, vec_ok, terms);
  if (e != cudaSuccess) return (int)e;
  if (partial) {
    int r = launch_splitk_reduce(stream, m, n, p.splits, partial, c, ldc, accumulate, epi, aux, ldaux);
    if (r) return r;
  }
  return 0;
}

int tc_clear() {
  const int zero = 0;
  return (int)cudaMemcpyToSymbol(g_tc_error, &zero, sizeof(int));
}

int tc_status(int* out) {
  int v = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int));
  if (e != cudaSuccess) return (int)e;
  *out = v;
  return 0;
}

}  // namespace gcnsa
