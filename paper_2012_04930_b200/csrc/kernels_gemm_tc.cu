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
// One CTA per SM walks its share of the work items (a 128 x BN tile, optionally
// one k-slice of it).  Warps 0 and 2 stream fp32 boxes of A and of B into two
// rings of shared memory with TMA: an operand whose K index is contiguous in
// memory arrives K-major (one 32 x rows box), one whose M / N index is
// contiguous arrives MN-major (32 x 32 boxes, one per 32 rows), so neither H W
// nor H^T Q needs a transposed copy.  Warps 4-11 split the operands: A goes
// from its landing slot into tensor memory as a hi and a lo part (the slot is
// free again at once, which is what keeps enough loads in flight), the lo part
// of B into the buffer beside B.  Warp 1 issues the MMAs - A_hi B_hi, A_hi B_lo,
// A_lo B_hi - into a TMEM accumulator, and warps 12-15 read the accumulator
// back, turn it through shared memory so that global accesses are
// row-contiguous, and apply the epilogue - while the other roles already work on
// the CTA's next item in a second accumulator buffer.  All
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
// warps: 0 loads A, 1 issues the MMAs (and owns tensor memory), 2 loads B, 3 idle, 4-11 split the operands (two
// groups of four: a warp may only touch the quarter warp % 4 of tensor memory's lanes), 12-15 run the epilogue
constexpr int kSplitWarp0 = 4, kSplitWarps = 8, kSplitGroups = 2, kEpiWarp0 = 12, kEpiWarps = 4;
constexpr int kThreads = 32 * (kEpiWarp0 + kEpiWarps);
constexpr int EPI_PITCH = 36;                               // floats per row of an epilogue patch
constexpr int EPI_BYTES = kEpiWarps * 32 * EPI_PITCH * 4;   // 18 KiB
constexpr int A_BYTES = BM * BK * 4;                        // 16 KiB
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

// D (tensor memory) (+)= A B^T with A in tensor memory (128 lanes = rows, one 32-bit column per k) and B through a
// shared-memory descriptor
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
// 32 consecutive columns of this thread's TMEM lane (lane quarter of the warp + lane id)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]),
      "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]),
      "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
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

// lo = x - hi with hi = x with its 13 low mantissa bits cleared (second buffer, same offsets: elementwise, so the
// swizzled position of an element is the same in both).  The first buffer keeps the raw fp32 words: kind::tf32
// reads the sign, exponent and upper 10 mantissa bits of each word, which is exactly hi, so rewriting it would only
// cost shared-memory bandwidth.  Measured: results equal with and without a masking store; the parity tests of the
// tensor-core path (2e-5 of max) would fail on a part that rounded instead (2^-12 per operand).
__device__ __forceinline__ void split_buffer(const uint8_t* hi_buf, uint8_t* lo_buf, int bytes, int t, int n_threads) {
#pragma unroll 4
  for (int i = t; i < bytes / 16; i += n_threads) {
    const uint4 x = reinterpret_cast<const uint4*>(hi_buf)[i];
    float4 l;
    l.x = __uint_as_float(x.x) - __uint_as_float(x.x & 0xFFFFE000u);
    l.y = __uint_as_float(x.y) - __uint_as_float(x.y & 0xFFFFE000u);
    l.z = __uint_as_float(x.z) - __uint_as_float(x.z & 0xFFFFE000u);
    l.w = __uint_as_float(x.w) - __uint_as_float(x.w & 0xFFFFE000u);
    reinterpret_cast<float4*>(lo_buf)[i] = l;
  }
}

// The shape of one kernel variant: tile width, operand layouts, and whether the accumulator is double-buffered.
//
// What bounds these products is how many bytes of the long operand a CTA keeps in flight from HBM (a ring of TMA
// boxes that only streams a 51 249 x 602 matrix reaches 2.6 / 3.3 / 3.5 / 3.9 TB/s with 32 / 48 / 64 / 96 KiB per
// SM), so the A operand has a landing ring of its own whose slots are free again as soon as the split warps have
// read them: they store the hi and the lo part of A into tensor memory (one lane per row, 32 + 32 columns per
// stage) and the MMAs read A from there.  Only B (with its lo part beside it) stays in shared memory until the MMAs
// of its k-block have retired.
//
// Tensor memory has 512 columns: four A stages take 256, the accumulators the rest.  Where 2 BN columns per
// accumulator buffer fit (64-column tiles; 128-column tiles when every CTA has a single item, so one buffer),
// A_hi [B_hi | B_lo] is ONE instruction of 2 BN columns into two accumulators that the epilogue adds, and with
// A_lo B_hi that makes two instructions per 8 k; otherwise the three products are three instructions into one
// accumulator.  Measured with clock64 around the issue loop: a 128 x 128 x 32 k-block takes the issuing thread about
// 800 clocks with two instructions per 8 k, the TF32 rate of the tensor pipe for its 3 x 128 x 128 x 32 products
// (about 2000 multiply-adds per clock and SM), and 1000 with three.
template <int BN_, bool A_MN_, bool B_MN_, bool DB_>
struct Shape {
  static constexpr int BN = BN_;
  static constexpr bool A_MN = A_MN_, B_MN = B_MN_, DB = DB_;
  static constexpr int B_BYTES = BN * BK * 4;
  static constexpr int NBUF = DB ? 2 : 1;                 // accumulator buffers
  static constexpr bool MERGED = BN == 64 || !DB;
  static constexpr int ACC_COLS = MERGED ? 2 * BN : BN;   // columns of one buffer
  static constexpr int NS = 4;                            // stages: A in tensor memory, B and B_lo in shared memory
  static constexpr int NA = BN == 64 ? 8 : 4;             // landing slots of A
  static constexpr int A_COL0 = NBUF * ACC_COLS;          // first column of the A stages in tensor memory
  static constexpr int USED_COLS = A_COL0 + NS * 64;
  static constexpr int TMEM_COLS = USED_COLS <= 128 ? 128 : (USED_COLS <= 256 ? 256 : 512);
  static constexpr int B_OFF = NA * A_BYTES;
  static constexpr int EPI_OFF = B_OFF + NS * 2 * B_BYTES;
  static constexpr int BAR_OFF = EPI_OFF + EPI_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 512 + 1024;  // + barriers + room to align the base to 1024 bytes
  static_assert(ACC_COLS <= 256, "one instruction covers at most 256 columns");
  static_assert(USED_COLS <= 512, "tensor memory has 512 columns");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
};

struct Work {
  int64_t m0, n0;
  int kb0, n_kb, z;
};
__device__ __forceinline__ Work decode_work(int w, int tiles_m, int tiles_n, int k_blocks, int kb_per_split, int bn) {
  Work k;
  const int nt = w % tiles_n, r = w / tiles_n;
  k.n0 = (int64_t)nt * bn;
  k.m0 = (int64_t)(r % tiles_m) * BM;
  k.z = r / tiles_m;
  k.kb0 = k.z * kb_per_split;
  k.n_kb = max(min(k_blocks, k.kb0 + kb_per_split) - k.kb0, 0);
  return k;
}

// One CTA per SM walks the work items (tile x k-slice) blockIdx.x, blockIdx.x + gridDim.x, ...; the rings and the
// accumulator buffers keep their phase across items, so that the loads, the split and the MMAs of item i + 1 run
// while warps 12-15 turn the accumulator of item i around.
template <class S>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tf32x3(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int64_t M, int64_t N,
            int k_blocks, int k_blocks_per_split, int tiles_m, int tiles_n, int total_work, float* __restrict__ c,
            int64_t ldc, int accumulate, int epi, const float* __restrict__ aux, int64_t ldaux,
            int64_t slice_stride, int vec_ok, int terms, float* __restrict__ colsum_partial,
            const float* __restrict__ post_scale) {
  constexpr int BN = S::BN, NS = S::NS, NA = S::NA, B_BYTES = S::B_BYTES;
  constexpr int ACC_COLS = S::ACC_COLS, NBUF = S::NBUF;
  constexpr bool A_MN = S::A_MN, B_MN = S::B_MN;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::BAR_OFF);
  uint64_t* full_a = bars;                     // A box landed                       (1 arrival + bytes)
  uint64_t* free_a = full_a + NA;              // A slot read by the split           (one arrival per warp of a group)
  uint64_t* full_b = free_a + NA;              // B box landed                       (1 arrival + bytes)
  uint64_t* split = full_b + NS;               // A in tensor memory, B_lo written   (one arrival per warp of a group)
  uint64_t* empty = split + NS;                // MMAs of the stage retired          (1 arrival by tcgen05.commit)
  uint64_t* acc_full = empty + NS;             // accumulator buffer complete        (1 arrival by tcgen05.commit)
  uint64_t* acc_empty = acc_full + NBUF;       // accumulator buffer read back       (one arrival per epilogue warp)
  uint64_t* drain = acc_empty + NBUF;          // wind-down only: the MMAs issued before a failed wait have retired
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  int* abort_slot = reinterpret_cast<int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // a wait ran out in an earlier launch or in another CTA of this one: nothing is allocated, nothing is computed
  if (threadIdx.x == 0) *abort_slot = tc_error_now();
  __syncthreads();
  if (*abort_slot != 0) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < NA; ++i) {
      mbar_init(&full_a[i], 1);
      mbar_init(&free_a[i], kSplitWarps / kSplitGroups);
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_b[i], 1);
      mbar_init(&split[i], kSplitWarps / kSplitGroups);
      mbar_init(&empty[i], 1);
    }
    for (int b = 0; b < NBUF; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], kEpiWarps);
    }
    mbar_init(drain, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(S::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == 2) {
    // ---------------- TMA producers: warp 0 streams A, warp 2 streams B ----------------
    if (lane == 0) {
      const bool is_a = warp == 0;
      const uint32_t ring = is_a ? NA : NS;
      uint64_t* full = is_a ? full_a : full_b;
      uint64_t* freed = is_a ? free_a : empty;
      uint32_t g = 0;  // k-blocks issued so far, over all items
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_work; w += gridDim.x) {
        const Work wk = decode_work(w, tiles_m, tiles_n, k_blocks, k_blocks_per_split, BN);
        for (int it = 0; it < wk.n_kb; ++it, ++g) {
          const uint32_t s = g % ring, ph = (g / ring) & 1;
          ok = mbar_wait(&freed[s], ph ^ 1, is_a ? 1 : 2);
          if (!ok) break;
          const int kx = (wk.kb0 + it) * BK;
          if (is_a) {
            uint8_t* dst = smem + s * A_BYTES;
            mbar_expect_tx(&full[s], A_BYTES);
            if (A_MN) {
#pragma unroll
              for (int j = 0; j < BM / 32; ++j) tma_load_2d(dst + j * 4096, &map_a, (int)wk.m0 + 32 * j, kx, &full[s]);
            } else {
              tma_load_2d(dst, &map_a, kx, (int)wk.m0, &full[s]);
            }
          } else {
            uint8_t* dst = smem + S::B_OFF + s * 2 * B_BYTES;
            mbar_expect_tx(&full[s], B_BYTES);
            if (B_MN) {
#pragma unroll
              for (int j = 0; j < BN / 32; ++j) tma_load_2d(dst + j * 4096, &map_b, (int)wk.n0 + 32 * j, kx, &full[s]);
            } else {
              tma_load_2d(dst, &map_b, kx, (int)wk.n0, &full[s]);
            }
          }
        }
      }
      if (!ok || tc_error_now() != 0) {  // wind down: let the copies already issued land before the CTA exits
        const long long t0 = clock64();
        for (uint32_t gi = g > ring ? g - ring : 0; gi < g; ++gi) {
          uint64_t* b = &full[gi % ring];
          const uint32_t ph = (gi / ring) & 1;
          while (!mbar_try_wait(b, ph) && clock64() - t0 < kSpinCycles) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // instruction descriptor: D fp32, A (tensor memory) and B tf32, B K-major or MN-major, N x 128
      const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      const uint32_t idesc2 = (idesc & ~(0x3Fu << 17)) | ((uint32_t)((2 * BN) >> 3) << 17);  // the same with 2 BN columns
      uint32_t g = 0, item = 0;
      bool ok = true, issued = false;
      for (int w = blockIdx.x; ok && w < total_work; w += gridDim.x, ++item) {
        const Work wk = decode_work(w, tiles_m, tiles_n, k_blocks, k_blocks_per_split, BN);
        const uint32_t ab = item % NBUF, aph = (item / NBUF) & 1;
        ok = mbar_wait(&acc_empty[ab], aph ^ 1, 6);  // the epilogue has read this buffer's previous item back
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d = tmem_base + ab * ACC_COLS;
        for (int it = 0; it < wk.n_kb; ++it, ++g) {
          const uint32_t s = g % NS, ph = (g / NS) & 1;
          ok = mbar_wait(&split[s], ph, 3);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t base = smem_u32(smem + S::B_OFF + s * 2 * B_BYTES);
          const uint64_t b_hi = B_MN ? umma_desc_mn(base) : umma_desc(base);
          const uint64_t b_lo = B_MN ? umma_desc_mn(base + B_BYTES) : umma_desc(base + B_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 8; ++k) {
            // one MMA covers 8 k: 8 columns of A; in B 32 bytes further inside the swizzle atom (K-major) or the next
            // 1024-byte group (MN-major)
            const uint64_t adv_b = (uint64_t)((B_MN ? k * 1024 : k * 32) >> 4);
            const uint32_t first = (it | k) != 0;
            const uint32_t ta = tmem_base + (uint32_t)(S::A_COL0 + s * 64 + 8 * k);
            if (terms != 3) {
              umma_tf32_ta(d, ta, b_hi + adv_b, idesc, first);       // plain TF32: the leading parts only
            } else if constexpr (S::MERGED) {
              umma_tf32_ta(d, ta, b_hi + adv_b, idesc2, first);      // A_hi [B_hi | B_lo]
              umma_tf32_ta(d, ta + 32, b_hi + adv_b, idesc, 1);      // + A_lo B_hi on the first half
            } else {
              umma_tf32_ta(d, ta, b_hi + adv_b, idesc, first);
              umma_tf32_ta(d, ta, b_lo + adv_b, idesc, 1);
              umma_tf32_ta(d, ta + 32, b_hi + adv_b, idesc, 1);
            }
          }
          umma_commit(&empty[s]);  // arrives when the MMAs above have finished reading this stage
          issued = true;
        }
        if (!ok) break;
        umma_commit(&acc_full[ab]);
      }
      if (!ok && issued) {
        // a wait ran out: the MMAs issued so far must have retired before the accumulator columns are given back
        umma_commit(drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(drain, 0) && clock64() - t0 < kSpinCycles) {
        }
      }
    }
  } else if (warp >= kSplitWarp0 && warp < kSplitWarp0 + kSplitWarps) {
    // ---------------- operand split (warps 4..11): group 0 takes the even k-blocks, group 1 the odd ones ----------
    // thread = row 32 q + lane of the A tile (q = the lane quarter of tensor memory this warp may touch)
    const int q = warp & 3, group = (warp - kSplitWarp0) >> 2, row = 32 * q + lane;
    const int tg = row;  // index among the 128 threads of the group
    uint32_t g = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok && w < total_work; w += gridDim.x) {
      const Work wk = decode_work(w, tiles_m, tiles_n, k_blocks, k_blocks_per_split, BN);
      for (int it = 0; it < wk.n_kb; ++it, ++g) {
        if ((int)(g % kSplitGroups) != group) continue;
        const uint32_t sa = g % NA, pa = (g / NA) & 1, s = g % NS, ps = (g / NS) & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(&full_a[sa], pa, 4));  // the warp gives up as a whole
        if (!ok) break;
        uint32_t v[32];
        const uint8_t* slot = smem + sa * A_BYTES;
        if (A_MN) {
          // four unswizzled boxes of 32 k x 32 rows: the 32 rows of one k are contiguous, a warp reads 128 bytes
          const uint8_t* p = slot + q * 4096 + lane * 4;
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = *reinterpret_cast<const uint32_t*>(p + k * 128);
        } else {
          // 128-byte swizzle: the 16-byte chunk c of row r sits at chunk position c ^ (r % 8)
          const uint8_t* arow = slot + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) {
            const uint4 x = *reinterpret_cast<const uint4*>(arow + ((cc ^ (row & 7)) << 4));
            v[4 * cc + 0] = x.x; v[4 * cc + 1] = x.y; v[4 * cc + 2] = x.z; v[4 * cc + 3] = x.w;
          }
        }
        // the stage (A columns in tensor memory, B_lo) is free once its B box has been loaded: that load waited for
        // the MMAs of the stage's previous k-block
        ok = __all_sync(0xffffffffu, mbar_wait(&full_b[s], ps, 7));
        if (!ok) break;
        const uint32_t ta = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(S::A_COL0 + s * 64);
        tmem_st32(ta, v);  // the raw words: the tensor core reads their leading 19 bits
        if (terms == 3) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) - __uint_as_float(v[j] & 0xFFFFE000u));
          tmem_st32(ta + 32, v);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&free_a[sa]);  // the landing slot can take the next box
        if (terms == 3) {
          uint8_t* bs = smem + S::B_OFF + s * 2 * B_BYTES;
          split_buffer(bs, bs + B_BYTES, B_BYTES, tg, 32 * kSplitWarps / kSplitGroups);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(&split[s]);
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ---------------- epilogue (warps 12..15) ----------------
    // A warp owns the 32 rows of its lane quarter of tensor memory and walks the tile's columns 32 at a time: read
    // back with thread = row, turned through a 32 x 32 patch of shared memory, stored with 8 lanes per row (128
    // contiguous bytes), 4 rows per instruction.
    const int quad = warp & 3;
    float* tile = reinterpret_cast<float*>(smem + S::EPI_OFF) + (warp - kEpiWarp0) * (32 * EPI_PITCH);
    const int lr = lane >> 3, lc = (lane & 7) * 4;
    const bool use_vec = vec_ok;
    const bool masked = use_vec && epi == GCNSA_EPI_MASK;
    const bool scale_here = epi == GCNSA_EPI_ROWSCALE;
    const int epi_l = scale_here ? GCNSA_EPI_NONE : epi;
    const int64_t n_pad = min(ldc, (N + 3) / 4 * 4);  // C's pad columns [N, n_pad) are written as zeros
    uint32_t item = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x, ++item) {
      const Work wk = decode_work(w, tiles_m, tiles_n, k_blocks, k_blocks_per_split, BN);
      const uint32_t ab = item % NBUF, aph = (item / NBUF) & 1;
      const int64_t row_base = wk.m0 + quad * 32;
      float* const cz = c + (int64_t)wk.z * slice_stride;  // k-slices write slices of a partial buffer shaped like C
      // the ReLU mask of the next 32 columns is fetched one step ahead (the first before the accumulator is
      // complete), so that its latency is not paid once per column step
      float4 mk[8];
      auto load_mask = [&](int c0) {
        const int64_t cm = wk.n0 + c0 + lc;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int64_t row = row_base + lr + 4 * i;
          mk[i] = (row < M && cm < n_pad) ? __ldg(reinterpret_cast<const float4*>(aux + row * ldaux + cm))
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      };
      if (masked) load_mask(0);
      // fused column sums: afterwards the rows are scaled (the next sparse product reads diag(s) G)
      float ps[8];
      if (colsum_partial && post_scale) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int64_t row = row_base + lr + 4 * i;
          ps[i] = row < M ? __ldg(post_scale + row) : 0.f;
        }
      }
      // a row scale is applied where a thread holds one row of the accumulator: one load per thread and tile
      float row_scale = 1.f;
      if (scale_here) {
        const int64_t my_row = row_base + lane;
        row_scale = my_row < M ? __ldg(aux + my_row) : 0.f;
      }
      bool ok = mbar_wait(&acc_full[ab], aph, 5);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t acc = tmem_base + ((uint32_t)(quad * 32) << 16) + ab * ACC_COLS;
      // steps of 32 columns; a step wholly outside C is not taken (C's zeroed pad columns end with N's step)
      const int last_c0 = (((int)min((int64_t)BN, N - wk.n0) + 31) / 32 - 1) * 32;
#pragma unroll 1
      for (int c0 = 0; c0 <= last_c0; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(acc + (uint32_t)c0, v);
        if constexpr (S::MERGED) {
          if (terms == 3) {  // the second accumulator: A_hi B_lo
            uint32_t u[32];
            tmem_ld32(acc + (uint32_t)(BN + c0), u);
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(u[j]));
          }
        }
        if (c0 == last_c0) {  // the accumulator is in registers: the MMAs of the next item may overwrite it
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        if (scale_here) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * row_scale);
        }
#pragma unroll
        for (int j = 0; j < 32; j += 4)  // thread = row; the pitch of 36 floats spreads 8 rows over all banks
          *reinterpret_cast<uint4*>(tile + lane * EPI_PITCH + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        uint32_t bits = 0;
        if (masked) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            bits |= ((mk[i].x > 0.f ? 1u : 0u) | (mk[i].y > 0.f ? 2u : 0u) | (mk[i].z > 0.f ? 4u : 0u) |
                     (mk[i].w > 0.f ? 8u : 0u))
                    << (4 * i);
          if (c0 < last_c0) load_mask(c0 + 32);
        }
        __syncwarp();
        const int64_t col = wk.n0 + c0 + lc;
        const unsigned vec_lanes = __ballot_sync(0xffffffffu, use_vec && col < n_pad);
        if (use_vec && col < n_pad) {
          // col is a multiple of 4 below n_pad, so at least one of the four columns is inside C; the float4 that
          // straddles N keeps `keep` of them, its other lanes are pad columns of the row (zeros)
          const int keep = (int)min((int64_t)4, N - col);
          float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if ((epi_l == GCNSA_EPI_BIAS || epi_l == GCNSA_EPI_BIAS_RELU) && aux) {
            if (keep == 4) {
              b4 = __ldg(reinterpret_cast<const float4*>(aux + col));
            } else {  // the bias has N entries
              b4.x = __ldg(aux + col);
              if (keep > 1) b4.y = __ldg(aux + col + 1);
              if (keep > 2) b4.z = __ldg(aux + col + 2);
            }
          }
          float4 a4[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) a4[i] = *reinterpret_cast<const float4*>(tile + (lr + 4 * i) * EPI_PITCH + lc);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (masked) {
              const uint32_t b = bits >> (4 * i);
              a4[i].x = (b & 1u) ? a4[i].x : 0.f; a4[i].y = (b & 2u) ? a4[i].y : 0.f;
              a4[i].z = (b & 4u) ? a4[i].z : 0.f; a4[i].w = (b & 8u) ? a4[i].w : 0.f;
            } else if (epi_l == GCNSA_EPI_BIAS || epi_l == GCNSA_EPI_BIAS_RELU) {
              a4[i].x += b4.x; a4[i].y += b4.y; a4[i].z += b4.z; a4[i].w += b4.w;
              if (epi_l == GCNSA_EPI_BIAS_RELU) {
                a4[i].x = fmaxf(a4[i].x, 0.f); a4[i].y = fmaxf(a4[i].y, 0.f);
                a4[i].z = fmaxf(a4[i].z, 0.f); a4[i].w = fmaxf(a4[i].w, 0.f);
              }
            }
          }
          if (keep < 4) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              if (keep < 2) a4[i].y = 0.f;
              if (keep < 3) a4[i].z = 0.f;
              a4[i].w = 0.f;
            }
          }
          if (colsum_partial) {
            // column sums of this warp's 32 rows (rows past M are zero rows of A, so they add nothing): the
            // thread's 8 rows, then the 4 threads that share these columns; one row of partial sums per warp
            float4 cs = a4[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) { cs.x += a4[i].x; cs.y += a4[i].y; cs.z += a4[i].z; cs.w += a4[i].w; }
#pragma unroll
            for (int o = 8; o <= 16; o <<= 1) {
              cs.x += __shfl_xor_sync(vec_lanes, cs.x, o); cs.y += __shfl_xor_sync(vec_lanes, cs.y, o);
              cs.z += __shfl_xor_sync(vec_lanes, cs.z, o); cs.w += __shfl_xor_sync(vec_lanes, cs.w, o);
            }
            if (lr == 0)
              *reinterpret_cast<float4*>(colsum_partial + ((wk.m0 / BM) * 4 + quad) * n_pad + col) = cs;
            if (post_scale) {
#pragma unroll
              for (int i = 0; i < 8; ++i) { a4[i].x *= ps[i]; a4[i].y *= ps[i]; a4[i].z *= ps[i]; a4[i].w *= ps[i]; }
            }
          }
          if (accumulate) {  // pad columns: what is there + 0
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int64_t row = row_base + lr + 4 * i;
              if (row < M) {
                const float4 o = *reinterpret_cast<const float4*>(cz + row * ldc + col);
                a4[i].x += o.x; a4[i].y += o.y; a4[i].z += o.z; a4[i].w += o.w;
              }
            }
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int64_t row = row_base + lr + 4 * i;
            if (row < M) *reinterpret_cast<float4*>(cz + row * ldc + col) = a4[i];
          }
        } else {
          for (int r = lr; r < 32; r += 4) {
            const int64_t row = row_base + r;
            if (row >= M) break;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int64_t cc = col + e;
              const float a = tile[r * EPI_PITCH + lc + e];
              if (cc < N) {
                const float o = epi_apply(a, epi_l, aux, ldaux, row, cc);
                float* dst = cz + row * ldc + cc;
                *dst = accumulate ? *dst + o : o;
              } else if (cc < n_pad && !accumulate) {
                cz[row * ldc + cc] = 0.f;
              }
            }
          }
        }
        __syncwarp();  // the patch is rewritten by the next step
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S::TMEM_COLS) : "memory");
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
// zero fill outside.  K-major operand: inner = k, outer = rows, box_outer = tile rows, 128-byte swizzle.
// MN-major operand: inner = rows (M or N), outer = k, box_outer = 32; B with the 128-byte swizzle of 32-byte atoms
// (the layout the tensor core transposes), A without swizzle (only the split warps read it).
enum class MapKind { kMajor, mnMajorSwizzled, mnMajorPlain };
bool make_map(CUtensorMap* map, const float* base, int64_t outer, int64_t inner, int64_t ld, int box_outer, MapKind kind) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = kind == MapKind::kMajor            ? CU_TENSOR_MAP_SWIZZLE_128B
                                : kind == MapKind::mnMajorSwizzled ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                                                                   : CU_TENSOR_MAP_SWIZZLE_NONE;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcPlan {
  int bn, splits, k_blocks, kb_per_split;
  size_t partial_bytes;
};

int sm_count() {
  static int n = 0;
  static std::once_flag once;
  std::call_once(once, [] {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  });
  return n;
}

TcPlan tc_plan(int64_t m, int64_t n, int64_t k) {
  TcPlan p;
  p.k_blocks = (int)((k + BK - 1) / BK);
  p.bn = n <= 64 ? 64 : 128;
  const int64_t tiles = ((m + BM - 1) / BM) * ((n + p.bn - 1) / p.bn);
  int64_t splits = 1;
  // few tiles with a long inner dimension: k-slices, so that the tiles' slices together fill the SMs once (5 tiles x
  // 30 slices would leave two work items for a second pass that takes as long as the first)
  const int sms = sm_count();
  if (tiles < sms / 2 && p.k_blocks >= 16) splits = std::min<int64_t>(sms / tiles, p.k_blocks / 8);
  splits = std::max<int64_t>(splits, 1);
  p.kb_per_split = (int)((p.k_blocks + splits - 1) / splits);
  p.splits = (p.k_blocks + p.kb_per_split - 1) / p.kb_per_split;
  if (p.splits < 1) p.splits = 1;
  auto up = [](size_t b) { return (b + 255) / 256 * 256; };
  // the k-slices' partial results: [splits][m][n rounded up to 4] (rows that take 16-byte stores)
  p.partial_bytes = up(p.splits > 1 ? (size_t)p.splits * m * ((n + 3) / 4 * 4) * sizeof(float) : 0);
  return p;
}

template <class S>
cudaError_t run_tc_shape(cudaStream_t s, const TcPlan& p, const CUtensorMap& ma, const CUtensorMap& mb, int64_t m,
                         int64_t n, int tiles_m, int tiles_n, int total, int grid, float* c, int64_t ldc, int accumulate,
                         int epi, const float* aux, int64_t ldaux, int64_t slice_stride, int vec_ok, int terms, float* colsum_partial, const float* post_scale) {
  cudaError_t e0 = cudaFuncSetAttribute(gemm_tf32x3<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::SMEM_BYTES);
  if (e0 != cudaSuccess) return e0;
  gemm_tf32x3<S><<<grid, kThreads, S::SMEM_BYTES, s>>>(ma, mb, m, n, p.k_blocks, p.kb_per_split, tiles_m, tiles_n, total,
                                                       c, ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
  note_launch();
  return cudaGetLastError();
}

template <int BN, bool A_MN, bool B_MN>
cudaError_t run_tc(cudaStream_t s, const TcPlan& p, const CUtensorMap& ma, const CUtensorMap& mb, int64_t m, int64_t n,
                   float* c, int64_t ldc, int accumulate, int epi, const float* aux, int64_t ldaux, int64_t slice_stride,
                   int vec_ok, int terms, float* colsum_partial, const float* post_scale) {
  const int64_t tiles_m = (m + BM - 1) / BM, tiles_n = (n + BN - 1) / BN;
  const int64_t total = tiles_m * tiles_n * p.splits;
  if (total >= (1LL << 31)) return cudaErrorInvalidValue;
  const int grid = (int)std::min<int64_t>(total, sm_count());
  // a second accumulator buffer pays only when a CTA has more than one work item
  if (total > grid)
    return run_tc_shape<Shape<BN, A_MN, B_MN, true>>(s, p, ma, mb, m, n, (int)tiles_m, (int)tiles_n, (int)total, grid, c,
                                                     ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
  return run_tc_shape<Shape<BN, A_MN, B_MN, false>>(s, p, ma, mb, m, n, (int)tiles_m, (int)tiles_n, (int)total, grid, c,
                                                    ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
}

template <int BN>
cudaError_t run_tc_major(bool a_mn, bool b_mn, cudaStream_t s, const TcPlan& p, const CUtensorMap& ma,
                         const CUtensorMap& mb, int64_t m, int64_t n, float* c, int64_t ldc, int accumulate, int epi,
                         const float* aux, int64_t ldaux, int64_t slice_stride, int vec_ok, int terms, float* colsum_partial, const float* post_scale) {
  if (a_mn && b_mn) return run_tc<BN, true, true>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
  if (a_mn) return run_tc<BN, true, false>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
  if (b_mn) return run_tc<BN, false, true>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
  return run_tc<BN, false, false>(s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, slice_stride, vec_ok, terms, colsum_partial, post_scale);
}

}  // namespace

// rows of column partial sums the fused epilogue writes: one per epilogue warp and row tile
int64_t gemm_tc_colsum_rows(int64_t m) { return (m + BM - 1) / BM * 4; }

size_t gemm_tc_workspace(int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k) {
  (void)ta; (void)tb;  // operands are read in the layout they have: no transposed copies to make room for
  return tc_plan(m, n, k).partial_bytes;
}

// Returns 0 on success, a cudaError_t on a CUDA failure, -1 when this shape / alignment / workspace cannot take
// the tensor-core path (the caller then uses the fp32 FMA kernel).
int launch_gemm_tc(void* stream, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a, int64_t lda,
                   const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi, const float* aux,
                   int64_t ldaux, void* workspace, size_t workspace_bytes, int terms, float* colsum_partial,
                   const float* post_scale) {
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
  const bool ok_a = a_mn ? make_map(&ma, a, k, m, lda, 32, MapKind::mnMajorPlain) : make_map(&ma, a, m, k, lda, BM, MapKind::kMajor);
  const bool ok_b = b_mn ? make_map(&mb, b, k, n, ldb, 32, MapKind::mnMajorSwizzled) : make_map(&mb, b, n, k, ldb, p.bn, MapKind::kMajor);
  if (!ok_a || !ok_b) return (int)cudaErrorInvalidValue;
  // float4 epilogue: C (and a mask) 16-byte aligned with pitches that are multiples of 4; a bias only needs alignment
  int vec_ok = (((uintptr_t)c & 15) == 0) && (ldc % 4 == 0);
  if (epi == GCNSA_EPI_MASK) vec_ok = vec_ok && (((uintptr_t)aux & 15) == 0) && (ldaux % 4 == 0);
  // the fused column sums exist in the float4 epilogue of unsliced products only
  if (colsum_partial && (!vec_ok || p.splits > 1 || ((uintptr_t)colsum_partial & 15))) return -1;
  if ((epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_BIAS_RELU) && aux) vec_ok = vec_ok && (((uintptr_t)aux & 15) == 0);
  cudaError_t e;
  if (partial) {
    // every k-slice writes its own slice of the partial buffer, plain; the reduction applies accumulate and epilogue
    const int64_t ldp = (n + 3) / 4 * 4;
    e = p.bn == 64 ? run_tc_major<64>(a_mn, b_mn, s, p, ma, mb, m, n, partial, ldp, 0, GCNSA_EPI_NONE, nullptr, 0, m * ldp, 1, terms, nullptr, nullptr)
                   : run_tc_major<128>(a_mn, b_mn, s, p, ma, mb, m, n, partial, ldp, 0, GCNSA_EPI_NONE, nullptr, 0, m * ldp, 1, terms, nullptr, nullptr);
    if (e != cudaSuccess) return (int)e;
    return launch_splitk_reduce(stream, m, n, p.splits, partial, ldp, c, ldc, accumulate, epi, aux, ldaux);
  }
  e = p.bn == 64 ? run_tc_major<64>(a_mn, b_mn, s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, 0, vec_ok, terms, colsum_partial, post_scale)
                 : run_tc_major<128>(a_mn, b_mn, s, p, ma, mb, m, n, c, ldc, accumulate, epi, aux, ldaux, 0, vec_ok, terms, colsum_partial, post_scale);
  if (e != cudaSuccess) return (int)e;
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
