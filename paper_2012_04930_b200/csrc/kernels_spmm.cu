// Y = epi(A X) for a CSR matrix A and a row-major fp32 matrix X: the normalized
// adjacency product of the GCN layer (Section 4.1) and, over the transposed
// CSR, of its backward pass.  One warp per row; G lanes cooperate on one
// non-zero, each lane owning CH float4 column chunks, so 32 / G non-zeros are
// gathered at once and every gather of a feature row is one coalesced
// 16-byte-per-lane request.  No atomics: each output row has one writer.
#include <cuda_runtime.h>

#include "internal.h"

namespace gcnsa {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ void fma4(float4& acc, float a, const float4& x) {
  acc.x = fmaf(a, x.x, acc.x);
  acc.y = fmaf(a, x.y, acc.y);
  acc.z = fmaf(a, x.z, acc.z);
  acc.w = fmaf(a, x.w, acc.w);
}

template <int G, int CH>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
spmm_warp_row(int n_rows, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
              const float* __restrict__ val, const int32_t* __restrict__ order, const float* __restrict__ x,
              int64_t ldx, int nvec, int f, int epi, const float* __restrict__ aux, int64_t ldaux,
              float* __restrict__ y, int64_t ldy) {
  constexpr int NG = 32 / G;  // non-zeros gathered per step
  const int w = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (w >= n_rows) return;
  const int lane = threadIdx.x & 31;
  const int g = lane / G, gl = lane % G;
  const int row = order ? __ldg(order + w) : w;
  const int beg = __ldg(rowptr + row), end = __ldg(rowptr + row + 1);

  float4 acc[CH];
#pragma unroll
  for (int ch = 0; ch < CH; ++ch) acc[ch] = make_float4(0.f, 0.f, 0.f, 0.f);

  // software pipeline over chunks of 32 non-zeros: indices and values of the
  // next chunk are in flight while the current chunk's feature rows are gathered
  int c_next = 0;
  float v_next = 0.f;
  if (beg + lane < end) {
    c_next = __ldg(col + beg + lane);
    v_next = __ldg(val + beg + lane);
  }
  for (int k = beg; k < end; k += 32) {
    const int c = c_next;
    const float v = v_next;
    const int kn = k + 32 + lane;
    c_next = 0;
    v_next = 0.f;
    if (kn < end) {
      c_next = __ldg(col + kn);
      v_next = __ldg(val + kn);
    }
    const int cnt = min(32, end - k);
    if (cnt == 32) {
#pragma unroll
      for (int j = 0; j < G; ++j) {
        const int src = j * NG + g;
        const int cc = __shfl_sync(kFull, c, src);
        const float vv = __shfl_sync(kFull, v, src);
        const float4* xr = reinterpret_cast<const float4*>(x + (int64_t)cc * ldx);
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
          const int q = gl + ch * G;
          if (q < nvec) fma4(acc[ch], vv, __ldg(xr + q));
        }
      }
    } else {
      const int steps = (cnt + NG - 1) / NG;
      for (int j = 0; j < steps; ++j) {
        const int src = j * NG + g;
        const int cc = __shfl_sync(kFull, c, src & 31);
        const float vv = __shfl_sync(kFull, v, src & 31);
        if (src < cnt) {
          const float4* xr = reinterpret_cast<const float4*>(x + (int64_t)cc * ldx);
#pragma unroll
          for (int ch = 0; ch < CH; ++ch) {
            const int q = gl + ch * G;
            if (q < nvec) fma4(acc[ch], vv, __ldg(xr + q));
          }
        }
      }
    }
  }
  // fold the NG partial sums (fixed order: deterministic)
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
  if (g != 0) return;
#pragma unroll
  for (int ch = 0; ch < CH; ++ch) {
    const int q = gl + ch * G;
    if (q >= nvec) continue;
    float4 r = acc[ch];
    const int c0 = q * 4;
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
      const float4 mk = __ldg(reinterpret_cast<const float4*>(aux + (int64_t)row * ldaux) + q);
      r.x = mk.x > 0.f ? r.x : 0.f;
      r.y = mk.y > 0.f ? r.y : 0.f;
      r.z = mk.z > 0.f ? r.z : 0.f;
      r.w = mk.w > 0.f ? r.w : 0.f;
    }
    reinterpret_cast<float4*>(y + (int64_t)row * ldy)[q] = r;
  }
}

template <int G, int CH>
cudaError_t run(cudaStream_t s, int n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                const int32_t* order, const float* x, int64_t ldx, int nvec, int f, int epi, const float* aux,
                int64_t ldaux, float* y, int64_t ldy) {
  const int grid = (n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  spmm_warp_row<G, CH><<<grid, kWarpsPerBlock * 32, 0, s>>>(n_rows, rowptr, col, val, order, x, ldx, nvec, f, epi, aux,
                                                           ldaux, y, ldy);
  note_launch();
  return cudaGetLastError();
}

}  // namespace

int launch_spmm(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                const int32_t* order, const float* x, int64_t ldx, int32_t f, int32_t epi, const float* aux,
                int64_t ldaux, float* y, int64_t ldy) {
  if (n_rows == 0 || f == 0) return 0;
  cudaStream_t s = (cudaStream_t)stream;
  const int n = (int)n_rows;
  const int nvec_total = (f + 3) / 4;
  // column slabs of at most 5 x 32 float4 (640 floats) per launch
  for (int v0 = 0; v0 < nvec_total; v0 += 160) {
    const int nvec = min(160, nvec_total - v0);
    const float* xs = x + 4 * v0;
    float* ys = y + 4 * v0;
    const float* auxs = aux;
    if (aux) auxs = aux + 4 * v0;  // bias and mask are both indexed by column
    const int fs = min(f - 4 * v0, 4 * nvec);
    cudaError_t e;
#define GCNSA_SPMM(G, CH) e = run<G, CH>(s, n, rowptr, col, val, order, xs, ldx, nvec, fs, epi, auxs, ldaux, ys, ldy)
    if (nvec <= 1) GCNSA_SPMM(1, 1);
    else if (nvec <= 2) GCNSA_SPMM(2, 1);
    else if (nvec <= 4) GCNSA_SPMM(4, 1);
    else if (nvec <= 8) GCNSA_SPMM(8, 1);
    else if (nvec <= 16) GCNSA_SPMM(16, 1);
    else if (nvec <= 32) GCNSA_SPMM(32, 1);
    else if (nvec <= 64) GCNSA_SPMM(32, 2);
    else if (nvec <= 96) GCNSA_SPMM(32, 3);
    else if (nvec <= 128) GCNSA_SPMM(32, 4);
    else GCNSA_SPMM(32, 5);
#undef GCNSA_SPMM
    if (e != cudaSuccess) return (int)e;
  }
  return 0;
}

}  // namespace gcnsa
