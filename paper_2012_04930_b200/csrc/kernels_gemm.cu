// C = epi(op(A) op(B)) (+ C): the dense feature transform H W of the GCN layer
// (Section 4.1) and the gradient products H^T dT and dT W^T, in fp32 FMA on the
// CUDA cores.  Shared-memory tiles of BM x BN x 16, 256 threads, each thread a
// (BM/16) x (BN/16) register tile, double-buffered with register prefetch.
// Products whose output is small but whose inner dimension is the row count of
// a partition (H^T dT) are split along k over blockIdx.z into a workspace and
// summed in a fixed order by a second kernel: deterministic, no atomics.
#include <cuda_runtime.h>

#include <algorithm>

#include "internal.h"

namespace gcnsa {

namespace {

constexpr int BK = 16;
constexpr int kThreads = 256;

// four consecutive elements (r, c..c+3) of a row-major R x C matrix, zero outside
template <bool VEC>
__device__ __forceinline__ float4 load4(const float* __restrict__ base, int64_t ld, int64_t r, int64_t c, int64_t R,
                                        int64_t C) {
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  if (r >= R || c >= C) return o;
  const float* p = base + r * ld + c;
  if (VEC && c + 3 < C) return __ldg(reinterpret_cast<const float4*>(p));
  o.x = __ldg(p);
  if (c + 1 < C) o.y = __ldg(p + 1);
  if (c + 2 < C) o.z = __ldg(p + 2);
  if (c + 3 < C) o.w = __ldg(p + 3);
  return o;
}

__device__ __forceinline__ float apply_epi(float v, int epi, const float* __restrict__ aux, int64_t ldaux, int64_t i,
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

template <int BM, int BN, bool TA, bool TB, bool VEC>
__global__ void __launch_bounds__(kThreads)
gemm_tile(int64_t M, int64_t N, int64_t K, int64_t k_per_split, const float* __restrict__ a, int64_t lda,
          const float* __restrict__ b, int64_t ldb, float* __restrict__ c, int64_t ldc, int accumulate, int epi,
          const float* __restrict__ aux, int64_t ldaux, float* __restrict__ partial) {
  constexpr int TM = BM / 16, TN = BN / 16;
  constexpr int A_F4 = BM * BK / 4 / kThreads, B_F4 = BN * BK / 4 / kThreads;
  __shared__ __align__(16) float As[2][BK][BM + 4];
  __shared__ __align__(16) float Bs[2][BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const int64_t k_begin = (int64_t)blockIdx.z * k_per_split;
  const int64_t k_end = min(K, k_begin + k_per_split);

  float4 ra[A_F4], rb[B_F4];
  auto fetch = [&](int64_t k0) {
#pragma unroll
    for (int i = 0; i < A_F4; ++i) {
      const int q = tid + i * kThreads;
      if (!TA) {  // stored M x K: four consecutive k of one row
        const int row = q / (BK / 4), kq = (q % (BK / 4)) * 4;
        ra[i] = load4<VEC>(a, lda, m0 + row, k0 + kq, M, k_end);
      } else {    // stored K x M: four consecutive rows of one k
        const int kk = q / (BM / 4), i4 = (q % (BM / 4)) * 4;
        ra[i] = load4<VEC>(a, lda, k0 + kk, m0 + i4, k_end, M);
      }
    }
#pragma unroll
    for (int i = 0; i < B_F4; ++i) {
      const int q = tid + i * kThreads;
      if (!TB) {  // stored K x N
        const int kk = q / (BN / 4), j4 = (q % (BN / 4)) * 4;
        rb[i] = load4<VEC>(b, ldb, k0 + kk, n0 + j4, k_end, N);
      } else {    // stored N x K
        const int col = q / (BK / 4), kq = (q % (BK / 4)) * 4;
        rb[i] = load4<VEC>(b, ldb, n0 + col, k0 + kq, N, k_end);
      }
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int i = 0; i < A_F4; ++i) {
      const int q = tid + i * kThreads;
      if (!TA) {
        const int row = q / (BK / 4), kq = (q % (BK / 4)) * 4;
        As[buf][kq + 0][row] = ra[i].x;
        As[buf][kq + 1][row] = ra[i].y;
        As[buf][kq + 2][row] = ra[i].z;
        As[buf][kq + 3][row] = ra[i].w;
      } else {
        const int kk = q / (BM / 4), i4 = (q % (BM / 4)) * 4;
        *reinterpret_cast<float4*>(&As[buf][kk][i4]) = ra[i];
      }
    }
#pragma unroll
    for (int i = 0; i < B_F4; ++i) {
      const int q = tid + i * kThreads;
      if (!TB) {
        const int kk = q / (BN / 4), j4 = (q % (BN / 4)) * 4;
        *reinterpret_cast<float4*>(&Bs[buf][kk][j4]) = rb[i];
      } else {
        const int col = q / (BK / 4), kq = (q % (BK / 4)) * 4;
        Bs[buf][kq + 0][col] = rb[i].x;
        Bs[buf][kq + 1][col] = rb[i].y;
        Bs[buf][kq + 2][col] = rb[i].z;
        Bs[buf][kq + 3][col] = rb[i].w;
      }
    }
  };

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  int buf = 0;
  if (k_begin < k_end) {
    fetch(k_begin);
    stash(0);
  }
  __syncthreads();
  for (int64_t k0 = k_begin; k0 < k_end; k0 += BK) {
    const bool more = k0 + BK < k_end;
    if (more) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float fa[TM], fb[TN];
#pragma unroll
      for (int h = 0; h < TM / 4; ++h) {
        const float4 t = *reinterpret_cast<const float4*>(&As[buf][kk][h * 64 + ty * 4]);
        fa[h * 4 + 0] = t.x; fa[h * 4 + 1] = t.y; fa[h * 4 + 2] = t.z; fa[h * 4 + 3] = t.w;
      }
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const float4 t = *reinterpret_cast<const float4*>(&Bs[buf][kk][h * 64 + tx * 4]);
        fb[h * 4 + 0] = t.x; fb[h * 4 + 1] = t.y; fb[h * 4 + 2] = t.z; fb[h * 4 + 3] = t.w;
      }
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(fa[i], fb[j], acc[i][j]);
    }
    if (more) {
      stash(buf ^ 1);
      __syncthreads();
      buf ^= 1;
    }
  }

  // epilogue; the pad columns [N, round_up(N, 4)) of C are written as zeros
  const int64_t n_pad = min(ldc, (N + 3) / 4 * 4);
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t gi = m0 + (i / 4) * 64 + ty * 4 + (i % 4);
    if (gi >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t gj = n0 + (j / 4) * 64 + tx * 4 + (j % 4);
      if (partial) {
        if (gj < N) partial[((int64_t)blockIdx.z * M + gi) * N + gj] = acc[i][j];
      } else if (gj < N) {
        float v = apply_epi(acc[i][j], epi, aux, ldaux, gi, gj);
        float* dst = c + gi * ldc + gj;
        *dst = accumulate ? *dst + v : v;
      } else if (gj < n_pad && !accumulate) {
        c[gi * ldc + gj] = 0.f;
      }
    }
  }
}

// C (+)= epi(sum_z partial[z]), partial = [splits][M][ldp]; pad columns [N, n_pad) are written as zeros.  A block covers 32 outputs; its
// 8 thread groups each add every 8th slice in ascending z and the 8 sums are added in group order: fixed order.
__global__ void __launch_bounds__(256)
splitk_reduce(int64_t M, int64_t N, int64_t n_pad, int splits, const float* __restrict__ partial, int64_t ldp,
              float* __restrict__ c,
              int64_t ldc, int accumulate, int epi, const float* __restrict__ aux, int64_t ldaux) {
  __shared__ float sh[8][32];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  const int64_t idx = (int64_t)blockIdx.x * 32 + lane;
  const bool live = idx < M * n_pad;
  const int64_t i = live ? idx / n_pad : 0, j = live ? idx % n_pad : 0;
  float s = 0.f;
  if (live && j < N)
    for (int z = grp; z < splits; z += 8) s += partial[((int64_t)z * M + i) * ldp + j];
  sh[grp][lane] = s;
  __syncthreads();
  if (grp != 0 || !live) return;
  float* dst = c + i * ldc + j;
  if (j >= N) {
    if (!accumulate) *dst = 0.f;
    return;
  }
  float t = sh[0][lane];
#pragma unroll
  for (int q = 1; q < 8; ++q) t += sh[q][lane];
  t = apply_epi(t, epi, aux, ldaux, i, j);
  *dst = accumulate ? *dst + t : t;
}

struct Plan {
  int bm, bn, splits;
  int64_t k_per_split;
};

Plan make_plan(int64_t m, int64_t n, int64_t k) {
  Plan p;
  p.bm = 128;
  p.bn = n <= 64 ? 64 : 128;
  if (m <= 64) p.bm = 64;
  const int64_t tiles = ((m + p.bm - 1) / p.bm) * ((n + p.bn - 1) / p.bn);
  const int64_t target = 2 * 148;  // two resident CTAs on each of the 148 SMs
  int64_t splits = 1;
  if (tiles < target / 2 && k >= 2048) {
    splits = std::min<int64_t>((target + tiles - 1) / tiles, k / 512);
    splits = std::max<int64_t>(splits, 1);
  }
  int64_t kps = (k + splits - 1) / splits;
  kps = (kps + BK - 1) / BK * BK;  // keeps every split's first k a multiple of 16 (vector alignment)
  if (kps < BK) kps = BK;          // k = 0 (an empty partition as the inner dimension): one split, no k steps
  p.splits = (int)((k + kps - 1) / kps);
  if (p.splits < 1) p.splits = 1;
  p.k_per_split = kps;
  return p;
}

template <int BM, int BN>
cudaError_t dispatch(cudaStream_t s, const Plan& p, bool ta, bool tb, bool vec, int64_t m, int64_t n, int64_t k,
                     const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc, int accumulate,
                     int epi, const float* aux, int64_t ldaux, float* partial) {
  dim3 grid((unsigned)((n + BN - 1) / BN), (unsigned)((m + BM - 1) / BM), (unsigned)p.splits);
#define GCNSA_GEMM(TA, TB, V)                                                                                       \
  gemm_tile<BM, BN, TA, TB, V><<<grid, kThreads, 0, s>>>(m, n, k, p.k_per_split, a, lda, b, ldb, c, ldc, accumulate, \
                                                         epi, aux, ldaux, partial)
  if (vec) {
    if (!ta && !tb) GCNSA_GEMM(false, false, true);
    else if (ta && !tb) GCNSA_GEMM(true, false, true);
    else if (!ta && tb) GCNSA_GEMM(false, true, true);
    else GCNSA_GEMM(true, true, true);
  } else {
    if (!ta && !tb) GCNSA_GEMM(false, false, false);
    else if (ta && !tb) GCNSA_GEMM(true, false, false);
    else if (!ta && tb) GCNSA_GEMM(false, true, false);
    else GCNSA_GEMM(true, true, false);
  }
#undef GCNSA_GEMM
  note_launch();
  return cudaGetLastError();
}

}  // namespace

size_t gemm_workspace(int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k) {
  const Plan p = make_plan(m, n, k);
  size_t need = p.splits > 1 ? (size_t)p.splits * (size_t)m * (size_t)n * sizeof(float) : 0;
  if (mode != GCNSA_GEMM_FP32) need = std::max(need, gemm_tc_workspace(ta, tb, m, n, k));
  return need;
}

int launch_splitk_reduce(void* stream, int64_t m, int64_t n, int splits, const float* partial, int64_t ldp, float* c,
                         int64_t ldc,
                         int accumulate, int epi, const float* aux, int64_t ldaux) {
  const int64_t n_pad = std::min<int64_t>(ldc, (n + 3) / 4 * 4);
  const int64_t total = m * n_pad;
  splitk_reduce<<<(unsigned)((total + 31) / 32), 256, 0, (cudaStream_t)stream>>>(m, n, n_pad, splits, partial, ldp, c, ldc,
                                                                                  accumulate, epi, aux, ldaux);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_gemm(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a,
                int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi,
                const float* aux, int64_t ldaux, void* workspace, size_t workspace_bytes) {
  if (m == 0 || n == 0) return 0;
  if (mode != GCNSA_GEMM_FP32 && k > 0) {
    const int r = launch_gemm_tc(stream, ta, tb, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, workspace,
                                 workspace_bytes, mode == GCNSA_GEMM_TF32 ? 1 : 3);
    if (r >= 0) {  // done, or a CUDA error
      if (r == 0) note_gemm_path(true);
      return r;
    }
    note_gemm_path(false);  // -1 = shape / alignment / workspace not eligible: fp32 FMA below
  }
  cudaStream_t s = (cudaStream_t)stream;
  Plan p = make_plan(m, n, k);
  const size_t need = p.splits > 1 ? (size_t)p.splits * (size_t)m * (size_t)n * sizeof(float) : 0;
  if (need > workspace_bytes || (need && !workspace)) {  // not enough scratch: run unsplit
    p.splits = 1;
    p.k_per_split = (k + BK - 1) / BK * BK;
    if (p.k_per_split == 0) p.k_per_split = BK;
  }
  float* partial = p.splits > 1 ? (float*)workspace : nullptr;
  const bool vec = (lda % 4 == 0) && (ldb % 4 == 0) && ((uintptr_t)a % 16 == 0) && ((uintptr_t)b % 16 == 0);
  cudaError_t e;
  if (p.bm == 128 && p.bn == 128)
    e = dispatch<128, 128>(s, p, ta, tb, vec, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, partial);
  else if (p.bm == 128)
    e = dispatch<128, 64>(s, p, ta, tb, vec, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, partial);
  else if (p.bn == 128)
    e = dispatch<64, 128>(s, p, ta, tb, vec, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, partial);
  else
    e = dispatch<64, 64>(s, p, ta, tb, vec, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, partial);
  if (e != cudaSuccess) return (int)e;
  if (partial) {
    const int r = launch_splitk_reduce(stream, m, n, p.splits, partial, n, c, ldc, accumulate, epi, aux, ldaux);
    if (r) return r;
  }
  return 0;
}

// the rows of partial sums the product's epilogue writes (one per epilogue warp and row tile), 256-byte rounded
static size_t fused_partial_bytes(int64_t m, int32_t n) {
  return ((size_t)gemm_tc_colsum_rows(m) * (size_t)((n + 3) / 4 * 4) * sizeof(float) + 255) / 256 * 256;
}

// ... followed by the scratch of the column-sum kernels that add those rows up; or, when the product runs
// unfused, the scratch of the column sums over C itself
size_t gemm_colsum_scratch(int64_t m, int32_t n) {
  return std::max(fused_partial_bytes(m, n) + colsum_scratch(gemm_tc_colsum_rows(m), n), colsum_scratch(m, n));
}

int launch_gemm_mask_colsum(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k,
                            const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc,
                            const float* mask, int64_t ldmask, const float* row_scale, float* out, int32_t accumulate,
                            void* scratch, void* workspace, size_t workspace_bytes) {
  if (m == 0 || n == 0) return 0;
  if (mode != GCNSA_GEMM_FP32 && k > 0) {
    const int r = launch_gemm_tc(stream, ta, tb, m, n, k, a, lda, b, ldb, c, ldc, 0, GCNSA_EPI_MASK, mask, ldmask, workspace,
                                 workspace_bytes, mode == GCNSA_GEMM_TF32 ? 1 : 3, (float*)scratch, row_scale);
    if (r == 0) {
      note_gemm_path(true);
      // thousands of partial rows for a tall product: the column-sum kernels add them in their fixed order
      return launch_colsum(stream, gemm_tc_colsum_rows(m), n, (const float*)scratch, (n + 3) / 4 * 4, out, accumulate,
                           (uint8_t*)scratch + fused_partial_bytes(m, n));
    }
    if (r > 0) return r;
  }
  // the product on whichever kernel takes it, then one pass over C for the sums and the scaling
  const int r = launch_gemm(stream, mode, ta, tb, m, n, k, a, lda, b, ldb, c, ldc, 0, GCNSA_EPI_MASK, mask, ldmask, workspace,
                            workspace_bytes);
  if (r) return r;
  return launch_colsum_scaled(stream, m, n, c, ldc, out, accumulate, scratch, row_scale, row_scale ? c : nullptr, ldc);
}

}  // namespace gcnsa
