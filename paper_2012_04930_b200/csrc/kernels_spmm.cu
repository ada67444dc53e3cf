// Y = epi(A X) for a CSR matrix A and a row-major fp32 matrix X: the normalized
// adjacency product of the GCN layer (Section 4.1) and, over the transposed
// CSR, of its backward pass.
//
// One warp per row, rows issued longest class first (the caller's degree-sorted
// permutation); the first n_long rows of that permutation (hub rows of a
// power-law graph) get a whole thread block each.  The 32 lanes form 32 / G groups of G lanes; every group owns a
// contiguous slice of the row's non-zeros and every lane CH float4 column
// chunks, so one warp instruction gathers 32 / G feature rows with 16 bytes per
// lane.  With G < 32 column indices and values are read four at a time with
// 16-byte loads whose address is the same for all lanes of a group, U such quads
// ahead of the gathers; with G = 32 and stored values they are fetched coalesced,
// 32 at a time, and handed round through 128-byte slots of shared memory per warp.
// Each output row has one writer and a fixed summation order: no atomics,
// bitwise reproducible.
#include <cuda_runtime.h>

#include <algorithm>

#include "debug_check.h"
#include "internal.h"

namespace gcnsa {

namespace {

constexpr unsigned kFull = 0xffffffffu;

#if GCNSA_DBG
GCNSA_DBG_WORD(g_dbg_spmm);
// a gathered column index must name a row of the source matrix
#define GCNSA_CHECK_COLUMN(cc) \
  if (dbg.src_rows >= 0 && !dbg_in(&g_dbg_spmm, (cc), 0, dbg.src_rows, kDbgColumn)) return
// the bounds travel as an extra (by-value) parameter of the checking build's kernels and device functions
#define GCNSA_DBG_PARAM , const SpmmBounds dbg
#define GCNSA_DBG_ARG , dbg
#define GCNSA_DBG_LAUNCH_ARG , a.dbg
#else
#define GCNSA_CHECK_COLUMN(cc)
#define GCNSA_DBG_PARAM
#define GCNSA_DBG_ARG
#define GCNSA_DBG_LAUNCH_ARG
#endif

__device__ __forceinline__ void fma4(float4& acc, float a, const float4& x) {
  acc.x = fmaf(a, x.x, acc.x);
  acc.y = fmaf(a, x.y, acc.y);
  acc.z = fmaf(a, x.z, acc.z);
  acc.w = fmaf(a, x.w, acc.w);
}

__device__ __forceinline__ void add4(float4& acc, const float4& x) {
  acc.x += x.x;
  acc.y += x.y;
  acc.z += x.z;
  acc.w += x.w;
}

// Adds the non-zeros [beg, end) that fall into slice `slice` of `n_slices` equal quad ranges to acc.
// UNIT: every stored entry counts as 1 (the 0/1 pattern A + I); `val` is not read.
template <int G, int CH, int U, bool UNIT>
__device__ __forceinline__ void accumulate_slice(float4 (&acc)[CH], int beg, int end, int slice, int n_slices, int gl,
                                                 const int32_t* __restrict__ col, const float* __restrict__ val,
                                                 const float4* __restrict__ x, int64_t ldx4, int nvec, int vec_idx GCNSA_DBG_PARAM) {
  const float4* xl = x + gl;
  auto gather = [&](int cc, float vv) {
    GCNSA_CHECK_COLUMN(cc);
    const float4* xr = xl + (int64_t)cc * ldx4;
#pragma unroll
    for (int ch = 0; ch < CH; ++ch)
      if (gl + ch * G < nvec) {
        if (UNIT) add4(acc[ch], __ldg(xr + ch * G));
        else fma4(acc[ch], vv, __ldg(xr + ch * G));
      }
  };
  auto edge_quad = [&](int e0) {  // a quad that sticks out of [beg, end): element by element
    for (int t = 0; t < 4; ++t) {
      const int e = e0 + t;
      if (e >= beg && e < end) gather(__ldg(col + e), UNIT ? 1.f : __ldg(val + e));
    }
  };
  // quads are aligned to absolute multiples of 4 so that their loads are 16-byte aligned
  const int a0 = beg & ~3;
  const int nq = (end - a0 + 3) >> 2;
  const int qps = (nq + n_slices - 1) / n_slices;
  const int q0 = slice * qps, q1 = min(nq, q0 + qps);
  int q = q0;
  if (q < q1 && a0 + 4 * q < beg) {
    edge_quad(a0 + 4 * q);
    ++q;
  }
  const int qfull = vec_idx ? min(q1, (end - a0) >> 2) : q;  // quads that lie entirely below `end`
  for (; q + U <= qfull; q += U) {
    int4 c4[U];
    float4 v4[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      c4[u] = __ldg(reinterpret_cast<const int4*>(col + a0 + 4 * (q + u)));
      if (!UNIT) v4[u] = __ldg(reinterpret_cast<const float4*>(val + a0 + 4 * (q + u)));
      else v4[u] = make_float4(1.f, 1.f, 1.f, 1.f);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      gather(c4[u].x, v4[u].x);
      gather(c4[u].y, v4[u].y);
      gather(c4[u].z, v4[u].z);
      gather(c4[u].w, v4[u].w);
    }
  }
  for (; q < qfull; ++q) {
    const int4 c4 = __ldg(reinterpret_cast<const int4*>(col + a0 + 4 * q));
    const float4 v4 = UNIT ? make_float4(1.f, 1.f, 1.f, 1.f) : __ldg(reinterpret_cast<const float4*>(val + a0 + 4 * q));
    gather(c4.x, v4.x);
    gather(c4.y, v4.y);
    gather(c4.z, v4.z);
    gather(c4.w, v4.w);
  }
  for (; q < q1; ++q) edge_quad(a0 + 4 * q);
}

// The element range of slice `slice` of `n_slices` (the same cut into aligned quads as accumulate_slice makes).
__device__ __forceinline__ void slice_range(int beg, int end, int slice, int n_slices, int& e0, int& e1) {
  const int a0 = beg & ~3;
  const int nq = (end - a0 + 3) >> 2;
  const int qps = (nq + n_slices - 1) / n_slices;
  const int q0 = slice * qps, q1 = min(nq, q0 + qps);
  e0 = max(beg, a0 + 4 * q0);
  e1 = q0 < q1 ? min(end, a0 + 4 * q1) : e0;
}

// Whole-warp shapes (G = 32: every lane holds CH chunks of the same source row) that read stored values.  A
// warp-uniform 16-byte load of four indices or values costs the L1 data path four wavefronts, one per non-zero,
// next to the four of a 512-byte gather.  Here lane l fetches the index and value of non-zero base + l, one
// coalesced wavefront per 32 non-zeros, the warp parks them in its 128-byte slots of shared memory and reads them
// back four at a time as broadcasts; the fetch of the next 32 is in flight while the current 32 are gathered.
// Elements are added in index order, as in accumulate_slice.  (With unit entries only the indices are left to
// broadcast; there the uniform loads of accumulate_slice measured 1 % faster, so that path keeps them.)
template <int CH, bool UNIT>
__device__ __forceinline__ void accumulate_range_staged(float4 (&acc)[CH], int e0, int e1, int lane,
                                                        const int32_t* __restrict__ col, const float* __restrict__ val,
                                                        const float4* __restrict__ x, int64_t ldx4, int nvec,
                                                        int32_t* sidx, float* sval GCNSA_DBG_PARAM) {
  const float4* xl = x + lane;
  auto gather = [&](int cc, float vv) {
    GCNSA_CHECK_COLUMN(cc);
    const float4* xr = xl + (int64_t)cc * ldx4;
#pragma unroll
    for (int ch = 0; ch < CH; ++ch)
      if (lane + ch * 32 < nvec) {
        if (UNIT) add4(acc[ch], __ldg(xr + ch * 32));
        else fma4(acc[ch], vv, __ldg(xr + ch * 32));
      }
  };
  int nxt_c = 0;
  float nxt_v = 0.f;
  if (e0 + lane < e1) {
    nxt_c = __ldg(col + e0 + lane);
    if (!UNIT) nxt_v = __ldg(val + e0 + lane);
  }
  for (int base = e0; base < e1; base += 32) {
    __syncwarp();  // the reads of the previous 32 are done
    sidx[lane] = nxt_c;
    if (!UNIT) sval[lane] = nxt_v;
    __syncwarp();
    if (base + 32 + lane < e1) {
      nxt_c = __ldg(col + base + 32 + lane);
      if (!UNIT) nxt_v = __ldg(val + base + 32 + lane);
    }
    const int cnt = min(32, e1 - base);
    int k = 0;
#pragma unroll 4
    for (; k + 4 <= cnt; k += 4) {
      const int4 c4 = *reinterpret_cast<const int4*>(sidx + k);
      float4 v4 = make_float4(1.f, 1.f, 1.f, 1.f);
      if (!UNIT) v4 = *reinterpret_cast<const float4*>(sval + k);
      gather(c4.x, v4.x);
      gather(c4.y, v4.y);
      gather(c4.z, v4.z);
      gather(c4.w, v4.w);
    }
    for (; k < cnt; ++k) gather(sidx[k], UNIT ? 1.f : sval[k]);
  }
}

// Folds the 32 / G group sums of a warp (fixed order); afterwards the lanes of group 0 hold the warp's sum.
template <int G, int CH>
__device__ __forceinline__ void fold_groups(float4 (&acc)[CH]) {
#pragma unroll
  for (int off = G; off < 32; off <<= 1) {
#pragma unroll
    for (int ch = 0; ch < CH; ++ch) {
      acc[ch].x += __shfl_xor_sync(kFull, acc[ch].x, off);
      acc[ch].y += __shfl_xor_sync(kFull, acc[ch].y, off);
      acc[ch].z += __shfl_xor_sync(kFull, acc[ch].z, off);
      acc[ch].w += __shfl_xor_sync(kFull, acc[ch].w, off);
    }
  }
}

// Epilogue + store of float4 chunk qq of one output row.
__device__ __forceinline__ void store_chunk(float4 r, int row, int qq, int f, int epi, const float* __restrict__ aux,
                                            int64_t ldaux, float* __restrict__ y, int64_t ldy) {
  const int c0 = qq * 4;
  if (epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_BIAS_RELU) {
    if (aux) {
      r.x += (c0 + 0 < f) ? __ldg(aux + c0 + 0) : 0.f;
      r.y += (c0 + 1 < f) ? __ldg(aux + c0 + 1) : 0.f;
      r.z += (c0 + 2 < f) ? __ldg(aux + c0 + 2) : 0.f;
      r.w += (c0 + 3 < f) ? __ldg(aux + c0 + 3) : 0.f;
    }
    if (epi == GCNSA_EPI_BIAS_RELU) {
      r.x = fmaxf(r.x, 0.f);
      r.y = fmaxf(r.y, 0.f);
      r.z = fmaxf(r.z, 0.f);
      r.w = fmaxf(r.w, 0.f);
    }
  } else if (epi == GCNSA_EPI_MASK) {
    const float4 mk = __ldg(reinterpret_cast<const float4*>(aux + (int64_t)row * ldaux) + qq);
    r.x = mk.x > 0.f ? r.x : 0.f;
    r.y = mk.y > 0.f ? r.y : 0.f;
    r.z = mk.z > 0.f ? r.z : 0.f;
    r.w = mk.w > 0.f ? r.w : 0.f;
  }
  reinterpret_cast<float4*>(y + (int64_t)row * ldy)[qq] = r;
}

// Blocks [0, n_long): one thread block per long row order[b]; its TPB / 32 warps take equal parts of the row,
// their sums meet in shared memory and are added in warp order (fixed order), so a hub row of thousands of
// non-zeros is not one warp's serial chain.  Blocks after that: one warp per row order[n_long ..).  One launch,
// longest rows dispatched first.
template <int G, int CH, int U, int TPB, int MINB, bool UNIT>
__global__ void __launch_bounds__(TPB, MINB)
spmm_rows(int n_long, int n_rows, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
          const float* __restrict__ val, const float* __restrict__ rscale, const int32_t* __restrict__ order,
          const float4* __restrict__ x, int64_t ldx4,
          int nvec, int f, int vec_idx, int epi, const float* __restrict__ aux, int64_t ldaux, float* __restrict__ y,
          int64_t ldy GCNSA_DBG_PARAM) {
  constexpr int NG = 32 / G;
  constexpr int W = TPB / 32;
  __shared__ float4 part[W][G * CH];
  __shared__ __align__(16) int32_t stage_idx[(G == 32 && !UNIT) ? W : 1][32];
  __shared__ __align__(16) float stage_val[(G == 32 && !UNIT) ? W : 1][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane / G, gl = lane % G;
  float4 acc[CH];
#pragma unroll
  for (int ch = 0; ch < CH; ++ch) acc[ch] = make_float4(0.f, 0.f, 0.f, 0.f);

  if ((int)blockIdx.x < n_long) {
    const int row = __ldg(order + blockIdx.x);
#if GCNSA_DBG
    if (dbg.mat_rows >= 0 && !dbg_in(&g_dbg_spmm, row, 0, dbg.mat_rows, kDbgOrderEntry)) return;  // whole block alike
#endif
    const int beg = __ldg(rowptr + row), end = __ldg(rowptr + row + 1);
#if GCNSA_DBG
    if (!dbg_in(&g_dbg_spmm, beg, 0, (long long)end + 1, kDbgRowRange)) return;
    if (dbg.nnz >= 0 && !dbg_in(&g_dbg_spmm, end, 0, dbg.nnz + 1, kDbgRowRange)) return;
#endif
    if constexpr (G == 32 && !UNIT) {
      int e0, e1;
      slice_range(beg, end, warp, W, e0, e1);
      accumulate_range_staged<CH, UNIT>(acc, e0, e1, lane, col, val, x, ldx4, nvec, stage_idx[warp], stage_val[warp] GCNSA_DBG_ARG);
    } else {
      accumulate_slice<G, CH, U, UNIT>(acc, beg, end, warp * NG + g, W * NG, gl, col, val, x, ldx4, nvec, vec_idx GCNSA_DBG_ARG);
    }
    fold_groups<G, CH>(acc);
    if (g == 0) {
#pragma unroll
      for (int ch = 0; ch < CH; ++ch) part[warp][gl + ch * G] = acc[ch];
    }
    __syncthreads();
    if (warp != 0 || g != 0) return;
#pragma unroll
    for (int ch = 0; ch < CH; ++ch) {
      const int qq = gl + ch * G;
      if (qq >= nvec) continue;
      float4 r = part[0][qq];
#pragma unroll
      for (int k = 1; k < W; ++k) {
        const float4 t = part[k][qq];
        r.x += t.x; r.y += t.y; r.z += t.z; r.w += t.w;
      }
      if (rscale) {
        const float sc = __ldg(rscale + row);
        r.x *= sc; r.y *= sc; r.z *= sc; r.w *= sc;
      }
      store_chunk(r, row, qq, f, epi, aux, ldaux, y, ldy);
    }
    return;
  }
  const int w = n_long + ((int)blockIdx.x - n_long) * W + warp;
  if (w >= n_rows) return;
  const int row = order ? __ldg(order + w) : w;
#if GCNSA_DBG
  if (dbg.mat_rows >= 0 && !dbg_in(&g_dbg_spmm, row, 0, dbg.mat_rows, kDbgOrderEntry)) return;  // whole warp alike
#endif
  const int beg = __ldg(rowptr + row), end = __ldg(rowptr + row + 1);
#if GCNSA_DBG
  if (!dbg_in(&g_dbg_spmm, beg, 0, (long long)end + 1, kDbgRowRange)) return;
  if (dbg.nnz >= 0 && !dbg_in(&g_dbg_spmm, end, 0, dbg.nnz + 1, kDbgRowRange)) return;
#endif
  if constexpr (G == 32 && !UNIT) {
    accumulate_range_staged<CH, UNIT>(acc, beg, end, lane, col, val, x, ldx4, nvec, stage_idx[warp], stage_val[warp] GCNSA_DBG_ARG);
  } else {
    accumulate_slice<G, CH, U, UNIT>(acc, beg, end, g, NG, gl, col, val, x, ldx4, nvec, vec_idx GCNSA_DBG_ARG);
  }
  fold_groups<G, CH>(acc);
  if (g != 0) return;
  const float sc = rscale ? __ldg(rscale + row) : 1.f;
#pragma unroll
  for (int ch = 0; ch < CH; ++ch) {
    const int qq = gl + ch * G;
    if (qq >= nvec) continue;
    float4 r = acc[ch];
    if (rscale) { r.x *= sc; r.y *= sc; r.z *= sc; r.w *= sc; }
    store_chunk(r, row, qq, f, epi, aux, ldaux, y, ldy);
  }
}

struct Args {
  cudaStream_t s;
  int n_rows;
  const int32_t *rowptr, *col;
  const float* val;
  const float* rscale;
  const int32_t* order;
  int n_long;
  const float* x;
  int64_t ldx;
  int nvec, f, vec_idx, epi;
  const float* aux;
  int64_t ldaux;
  float* y;
  int64_t ldy;
  SpmmBounds dbg;
};

template <int G, int CH, int U, int TPB, int MINB>
cudaError_t run(const Args& a) {
  const int rows_per_block = TPB / 32;
  const int grid = a.n_long + (a.n_rows - a.n_long + rows_per_block - 1) / rows_per_block;
  if (a.val)
    spmm_rows<G, CH, U, TPB, MINB, false><<<grid, TPB, 0, a.s>>>(
        a.n_long, a.n_rows, a.rowptr, a.col, a.val, a.rscale, a.order, reinterpret_cast<const float4*>(a.x), a.ldx / 4,
        a.nvec, a.f, a.vec_idx, a.epi, a.aux, a.ldaux, a.y, a.ldy GCNSA_DBG_LAUNCH_ARG);
  else
    spmm_rows<G, CH, U, TPB, MINB, true><<<grid, TPB, 0, a.s>>>(
        a.n_long, a.n_rows, a.rowptr, a.col, nullptr, a.rscale, a.order, reinterpret_cast<const float4*>(a.x), a.ldx / 4,
        a.nvec, a.f, a.vec_idx, a.epi, a.aux, a.ldaux, a.y, a.ldy GCNSA_DBG_LAUNCH_ARG);
  note_launch();
  return cudaGetLastError();
}

}  // namespace

int launch_spmm(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                const float* row_scale, const int32_t* order, int64_t n_long, const float* x, int64_t ldx, int32_t f, int32_t epi, const float* aux,
                int64_t ldaux, float* y, int64_t ldy, const SpmmBounds& bounds) {
  if (n_rows == 0 || f == 0) return 0;
  Args a;
  a.dbg = bounds;
  a.s = (cudaStream_t)stream;
  a.n_rows = (int)n_rows;
  a.rowptr = rowptr; a.col = col; a.val = val; a.rscale = row_scale; a.order = order;
  a.n_long = order ? (int)std::min<int64_t>(std::max<int64_t>(n_long, 0), n_rows) : 0;
  a.ldx = ldx; a.epi = epi; a.ldaux = ldaux; a.ldy = ldy;
  // 16-byte index loads need 16-byte aligned arrays; otherwise every quad goes element by element
  a.vec_idx = (((uintptr_t)col | (uintptr_t)val) & 15) == 0 ? 1 : 0;  // val == NULL (unit entries) counts as aligned
  const int nvec_total = (f + 3) / 4;
  // column slabs of at most 5 x 32 float4 (640 floats) per launch
  for (int v0 = 0; v0 < nvec_total; v0 += 160) {
    a.nvec = min(160, nvec_total - v0);
    a.x = x + 4 * v0;
    a.y = y + 4 * v0;
    a.aux = aux ? aux + 4 * v0 : nullptr;  // bias and mask are both indexed by column
    a.f = min(f - 4 * v0, 4 * a.nvec);
    cudaError_t e;
    const int nv = a.nvec;
    // MINB (blocks per SM the register allocation must allow) is part of the tuning: the kernel is bound by the
    // L1 data path, and about 32-40 resident warps per SM (64 resp. 48 registers a thread) measured fastest;
    // left alone the compiler unrolls to over 100 registers (16 warps), and at 32 registers (64 warps) L1 thrashes.
    if (nv <= 4) e = run<4, 1, 2, 128, 10>(a);
    else if (nv <= 8) e = run<4, 2, 2, 128, 10>(a);
    else if (nv <= 12) e = run<4, 3, 2, 128, 10>(a);
    else if (nv <= 16) e = run<8, 2, 2, 128, 10>(a);
    else if (nv <= 32) e = run<32, 1, 4, 256, 4>(a);
    else if (nv <= 64) e = run<32, 2, 4, 256, 4>(a);
    else if (nv <= 96) e = run<32, 3, 2, 256, 3>(a);
    else if (nv <= 128) e = run<32, 4, 2, 256, 3>(a);
    else e = run<32, 5, 2, 256, 3>(a);
    if (e != cudaSuccess) return (int)e;
  }
  return 0;
}

int debug_word_spmm(unsigned long long* out, bool clear) {
  *out = 0ull;
#if GCNSA_DBG
  cudaError_t e = cudaMemcpyFromSymbol(out, g_dbg_spmm, sizeof(*out));
  if (e == cudaSuccess && clear) {
    const unsigned long long zero = 0ull;
    e = cudaMemcpyToSymbol(g_dbg_spmm, &zero, sizeof(zero));
  }
  return (int)e;
#else
  (void)clear;
  return 0;
#endif
}

}  // namespace gcnsa
