// Small memory-bound kernels of the training step: masked softmax
// cross-entropy (loss + gradient in one pass over the logits), bias gradient
// (column sums), gradient average + Adam, and the D^-1/2 (A+I) D^-1/2 weights.
// Reductions go through per-block partial sums that a second kernel adds in a
// fixed order: no floating-point atomics, results are run-to-run identical.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <mutex>

#include "internal.h"

namespace gcnsa {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kCeBlocksMax = 1184;  // 8 x 148
constexpr int kCeWarps = 8;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// One warp per row.  grad row = (softmax - onehot) * inv_nt for masked rows,
// zero otherwise; block partial of sum(lse - z_y) goes to partial[blockIdx.x].
__global__ void __launch_bounds__(kCeWarps * 32)
softmax_ce_rows(int64_t n, int c, const float* __restrict__ logits, int64_t ld, const int32_t* __restrict__ y,
                const uint8_t* __restrict__ mask, float inv_nt, float* __restrict__ grad, int64_t ldg,
                float* __restrict__ partial) {
  __shared__ float sh[kCeWarps];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int ldg_cols = (int)min(ldg, (int64_t)((c + 3) / 4 * 4));
  float loss = 0.f;
  for (int64_t row = (int64_t)blockIdx.x * kCeWarps + wib; row < n; row += (int64_t)gridDim.x * kCeWarps) {
    float* gr = grad + row * ldg;
    if (c <= 64) {
      // the row lives in two registers per lane; logits, label and mask are fetched together (no load waits for
      // another), the same sums in the same order as the general path below
      const float* z = logits + row * ld;
      const bool on = mask[row] != 0;
      const int yi = y[row];
      const int j0 = lane, j1 = lane + 32;
      const float z0 = j0 < c ? z[j0] : -INFINITY, z1 = j1 < c ? z[j1] : -INFINITY;
      if (!on) {
        for (int j = lane; j < ldg_cols; j += 32) gr[j] = 0.f;
        continue;
      }
      const float mx = warp_max(fmaxf(z0, z1));
      float se = 0.f;
      if (j0 < c) se += expf(z0 - mx);
      if (j1 < c) se += expf(z1 - mx);
      se = warp_sum(se);
      const float inv_se = 1.f / se;
      if (j0 < ldg_cols) gr[j0] = j0 < c ? (expf(z0 - mx) * inv_se - (j0 == yi ? 1.f : 0.f)) * inv_nt : 0.f;
      if (j1 < ldg_cols) gr[j1] = j1 < c ? (expf(z1 - mx) * inv_se - (j1 == yi ? 1.f : 0.f)) * inv_nt : 0.f;
      const float zy = __shfl_sync(kFull, yi < 32 ? z0 : z1, yi & 31);
      if (lane == 0) loss += (mx + logf(se)) - zy;
      continue;
    }
    if (!mask[row]) {
      for (int j = lane; j < ldg_cols; j += 32) gr[j] = 0.f;
      continue;
    }
    const float* z = logits + row * ld;
    float mx = -INFINITY;
    for (int j = lane; j < c; j += 32) mx = fmaxf(mx, z[j]);
    mx = warp_max(mx);
    float se = 0.f;
    for (int j = lane; j < c; j += 32) se += expf(z[j] - mx);
    se = warp_sum(se);
    const int yi = y[row];
    const float inv_se = 1.f / se;
    for (int j = lane; j < ldg_cols; j += 32) {
      float g = 0.f;
      if (j < c) g = (expf(z[j] - mx) * inv_se - (j == yi ? 1.f : 0.f)) * inv_nt;
      gr[j] = g;
    }
    if (lane == 0) loss += (mx + logf(se)) - z[yi];
  }
  if (lane == 0) sh[wib] = loss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < kCeWarps; ++i) s += sh[i];
    partial[blockIdx.x] = s;
  }
}

__global__ void loss_finalize(const float* __restrict__ partial, int count, float inv_nt, float* __restrict__ out) {
  __shared__ float sh[256];
  float s = 0.f;
  for (int i = threadIdx.x; i < count; i += 256) s += partial[i];
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = sh[0] * inv_nt;
}

__global__ void mean_kernel(const float* __restrict__ src, int count, float* __restrict__ dst) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < count; ++i) s += src[i];
    *dst = s / (float)count;
  }
}

// block (32, 8): x over columns, y over rows of the block's row range
__global__ void __launch_bounds__(256)
colsum_partial(int64_t n, int f, const float* __restrict__ g, int64_t ldg, int64_t rows_per_block,
               float* __restrict__ partial) {
  __shared__ float sh[8][33];
  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block, r1 = min(n, r0 + rows_per_block);
  for (int j0 = 0; j0 < f; j0 += 32) {
    const int j = j0 + threadIdx.x;
    float s = 0.f;
    if (j < f)
      for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) s += g[r * ldg + j];
    sh[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && j < f) {
      float t = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) t += sh[q][threadIdx.x];
      partial[(int64_t)blockIdx.x * f + j] = t;
    }
    __syncthreads();
  }
}

// Same sums for 16-byte aligned rows: thread (tx, ty) adds the float4 column chunk tx of rows ty, ty + RY, ...
// of the block's row range; the RY partial sums meet in shared memory and are added in ty order (fixed order).
// With `scaled` given the kernel also writes scaled[r, :] = rscale[r] * g[r, :] (whole float4 chunks; scaled may be
// g itself: every element is read once and then written by the same thread, with plain loads).
template <int NV>
__global__ void __launch_bounds__(256)
colsum_partial_v4(int64_t n, int f, const float* g, int64_t ldg, int64_t rows_per_block, float* __restrict__ partial,
                  const float* __restrict__ rscale, float* scaled, int64_t lds) {
  constexpr int RY = 256 / NV;
  __shared__ float4 sh[256];
  const int tx = threadIdx.x % NV, ty = threadIdx.x / NV;
  const int nvec = (f + 3) / 4;
  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block, r1 = min(n, r0 + rows_per_block);
  for (int v0 = 0; v0 < nvec; v0 += NV) {
    const int q = v0 + tx;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q < nvec) {
#pragma unroll 4
      for (int64_t r = r0 + ty; r < r1; r += RY) {
        const float4 t = *(reinterpret_cast<const float4*>(g + r * ldg) + q);
        acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        if (scaled) {
          const float sc = __ldg(rscale + r);
          reinterpret_cast<float4*>(scaled + r * lds)[q] = make_float4(sc * t.x, sc * t.y, sc * t.z, sc * t.w);
        }
      }
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    if (ty == 0 && q < nvec) {
      float4 t = sh[tx];
#pragma unroll
      for (int k = 1; k < RY; ++k) {
        const float4 u = sh[k * NV + tx];
        t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
      }
      float* dst = partial + (int64_t)blockIdx.x * f + 4 * q;
      dst[0] = t.x;
      if (4 * q + 1 < f) dst[1] = t.y;
      if (4 * q + 2 < f) dst[2] = t.z;
      if (4 * q + 3 < f) dst[3] = t.w;
    }
    __syncthreads();
  }
}

// out[j] (+)= sum over blocks of partial[b][j] (rows ldp floats apart).  A block covers 32 columns; its 8 thread groups add every 8th
// block's partial in ascending order and the 8 sums are added in group order: fixed order.
__global__ void __launch_bounds__(256)
colsum_final(int f, int blocks, const float* __restrict__ partial, int64_t ldp, float* __restrict__ out, int accumulate) {
  __shared__ float sh[8][32];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + lane;
  float s = 0.f;
  if (j < f)
    for (int b = grp; b < blocks; b += 8) s += partial[(int64_t)b * ldp + j];
  sh[grp][lane] = s;
  __syncthreads();
  if (grp != 0 || j >= f) return;
  float t = sh[0][lane];
#pragma unroll
  for (int q = 1; q < 8; ++q) t += sh[q][lane];
  out[j] = accumulate ? out[j] + t : t;
}

// Step counter and bias corrections kept on the device, so that a captured epoch can be replayed: state[0] = t
// (as a float-exact integer in a double), state[1] = 1 / (1 - beta1^t), state[2] = 1 / (1 - beta2^t).
__global__ void adam_advance(double* __restrict__ state, double b1, double b2) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const double t = state[0] + 1.0;
  state[0] = t;
  state[1] = 1.0 / (1.0 - pow(b1, t));
  state[2] = 1.0 / (1.0 - pow(b2, t));
}

__global__ void adam_kernel_dev(int64_t count, float* __restrict__ theta, float* __restrict__ gsum, float* __restrict__ m,
                                float* __restrict__ v, float inv_m, float lr, float b1, float b2, float eps,
                                const double* __restrict__ state) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float c1 = (float)state[1], c2 = (float)state[2];
  const float g = gsum[i] * inv_m;
  const float mi = b1 * m[i] + (1.f - b1) * g;
  const float vi = b2 * v[i] + (1.f - b2) * g * g;
  m[i] = mi;
  v[i] = vi;
  theta[i] -= lr * (mi * c1) / (sqrtf(vi * c2) + eps);
  gsum[i] = 0.f;
}

__global__ void adam_local_kernel_dev(int64_t count, const float* __restrict__ theta, float* __restrict__ gsum,
                                      float* __restrict__ m, float* __restrict__ v, float* __restrict__ acc, int first,
                                      float inv_m, float lr, float b1, float b2, float eps,
                                      const double* __restrict__ state) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float c1 = (float)state[1], c2 = (float)state[2];
  const float g = gsum[i];
  const float mi = b1 * m[i] + (1.f - b1) * g;
  const float vi = b2 * v[i] + (1.f - b2) * g * g;
  m[i] = mi;
  v[i] = vi;
  const float th = (theta[i] - lr * (mi * c1) / (sqrtf(vi * c2) + eps)) * inv_m;
  acc[i] = first ? th : acc[i] + th;
  gsum[i] = 0.f;
}

__global__ void adam_kernel(int64_t count, float* __restrict__ theta, float* __restrict__ gsum, float* __restrict__ m,
                            float* __restrict__ v, float inv_m, float lr, float b1, float b2, float eps, float c1,
                            float c2) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float g = gsum[i] * inv_m;
  const float mi = b1 * m[i] + (1.f - b1) * g;
  const float vi = b2 * v[i] + (1.f - b2) * g * g;
  m[i] = mi;
  v[i] = vi;
  // c1 = 1 / (1 - beta1^t), c2 = 1 / (1 - beta2^t)
  theta[i] -= lr * (mi * c1) / (sqrtf(vi * c2) + eps);
  gsum[i] = 0.f;
}

// one warp per row; hits[blockIdx.x] = number of masked rows of this block whose argmax equals the label
__global__ void __launch_bounds__(kCeWarps * 32)
argmax_hits_rows(int64_t n, int c, const float* __restrict__ logits, int64_t ld, const int32_t* __restrict__ y,
                 const uint8_t* __restrict__ mask, int32_t* __restrict__ pred, int32_t* __restrict__ hits) {
  __shared__ int sh[kCeWarps];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  int count = 0;
  for (int64_t row = (int64_t)blockIdx.x * kCeWarps + wib; row < n; row += (int64_t)gridDim.x * kCeWarps) {
    const float* z = logits + row * ld;
    float best = -INFINITY;
    int arg = 0x7fffffff;
    for (int j = lane; j < c; j += 32) {
      const float v = z[j];
      if (v > best) { best = v; arg = j; }   // strict: the first maximum of this lane's columns
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(kFull, best, o);
      const int oa = __shfl_xor_sync(kFull, arg, o);
      if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    if (lane == 0) {
      pred[row] = arg;
      if ((!mask || mask[row]) && arg == y[row]) ++count;
    }
  }
  if (lane == 0) sh[wib] = count;
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int i = 0; i < kCeWarps; ++i) s += sh[i];
    hits[blockIdx.x] = s;
  }
}

__global__ void __launch_bounds__(256)
normalize_rows(int64_t n_rows, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
               const int32_t* __restrict__ deg, float* __restrict__ val) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int lane = threadIdx.x & 31;
  const float di = (float)deg[row];
  for (int e = rowptr[row] + lane; e < rowptr[row + 1]; e += 32) val[e] = 1.0f / sqrtf(di * (float)deg[col[e]]);
}

int ce_blocks(int64_t n) { return (int)std::max<int64_t>(1, std::min<int64_t>((n + kCeWarps - 1) / kCeWarps, kCeBlocksMax)); }
int colsum_blocks(int64_t n) { return (int)std::max<int64_t>(1, std::min<int64_t>((n + 63) / 64, 296)); }

}  // namespace

size_t softmax_ce_scratch(int64_t n) { return (size_t)ce_blocks(n) * sizeof(float); }

int launch_softmax_ce(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                      const uint8_t* mask, int64_t n_train, float* loss_dev, float* grad, int64_t ldg, void* scratch) {
  cudaStream_t s = (cudaStream_t)stream;
  const int blocks = ce_blocks(n);
  const float inv_nt = n_train > 0 ? 1.0f / (float)n_train : 0.f;
  if (n > 0) {
    softmax_ce_rows<<<blocks, kCeWarps * 32, 0, s>>>(n, c, logits, ld, y, mask, inv_nt, grad, ldg, (float*)scratch);
    note_launch();
  }
  if (loss_dev) {
    loss_finalize<<<1, 256, 0, s>>>((const float*)scratch, n > 0 ? blocks : 0, inv_nt, loss_dev);
    note_launch();
  }
  return (int)cudaGetLastError();
}

size_t colsum_scratch(int64_t n, int32_t f) { return (size_t)colsum_blocks(n) * (size_t)f * sizeof(float); }

int launch_colsum(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                  void* scratch) {
  return launch_colsum_scaled(stream, n, f, g, ldg, out, accumulate, scratch, nullptr, nullptr, 0);
}

int launch_colsum_scaled(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                         void* scratch, const float* rscale, float* scaled, int64_t lds) {
  cudaStream_t s = (cudaStream_t)stream;
  const int blocks = colsum_blocks(n);
  const int64_t rpb = std::max<int64_t>(1, (n + blocks - 1) / blocks);
  const int nvec = (f + 3) / 4;
  const bool side = scaled != nullptr;
  const bool side_ok = !side || ((((uintptr_t)scaled & 15) == 0) && (lds % 4 == 0));
  if ((((uintptr_t)g & 15) == 0) && (ldg % 4 == 0) && side_ok) {
    float* p = (float*)scratch;
    if (nvec <= 8) colsum_partial_v4<8><<<blocks, 256, 0, s>>>(n, f, g, ldg, rpb, p, rscale, scaled, lds);
    else if (nvec <= 16) colsum_partial_v4<16><<<blocks, 256, 0, s>>>(n, f, g, ldg, rpb, p, rscale, scaled, lds);
    else if (nvec <= 32) colsum_partial_v4<32><<<blocks, 256, 0, s>>>(n, f, g, ldg, rpb, p, rscale, scaled, lds);
    else colsum_partial_v4<64><<<blocks, 256, 0, s>>>(n, f, g, ldg, rpb, p, rscale, scaled, lds);
  } else {
    // rows the vector kernel cannot take (unaligned base or pitch); the scaled side output exists in whole
    // float4 chunks only, so it cannot be produced for them
    if (side) return (int)cudaErrorMisalignedAddress;
    colsum_partial<<<blocks, dim3(32, 8), 0, s>>>(n, f, g, ldg, rpb, (float*)scratch);
  }
  colsum_final<<<(f + 31) / 32, 256, 0, s>>>(f, blocks, (const float*)scratch, f, out, accumulate);
  note_launch(2);
  return (int)cudaGetLastError();
}

int launch_adam(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m, float lr,
                float beta1, float beta2, float eps, int64_t t) {
  if (count == 0) return 0;
  const double c1 = 1.0 / (1.0 - std::pow((double)beta1, (double)t));
  const double c2 = 1.0 / (1.0 - std::pow((double)beta2, (double)t));
  adam_kernel<<<(unsigned)((count + 255) / 256), 256, 0, (cudaStream_t)stream>>>(count, theta, gsum, m, v, inv_m, lr,
                                                                                beta1, beta2, eps, (float)c1, (float)c2);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_adam_advance(void* stream, double* state, float beta1, float beta2) {
  adam_advance<<<1, 32, 0, (cudaStream_t)stream>>>(state, (double)beta1, (double)beta2);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_adam_dev(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m, float lr,
                    float beta1, float beta2, float eps, const double* state) {
  if (count == 0) return 0;
  adam_kernel_dev<<<(unsigned)((count + 255) / 256), 256, 0, (cudaStream_t)stream>>>(count, theta, gsum, m, v, inv_m, lr,
                                                                                    beta1, beta2, eps, state);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_adam_local_dev(void* stream, int64_t count, const float* theta, float* gsum, float* m, float* v, float* acc,
                          int first, float inv_m, float lr, float beta1, float beta2, float eps, const double* state) {
  if (count == 0) return 0;
  adam_local_kernel_dev<<<(unsigned)((count + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      count, theta, gsum, m, v, acc, first, inv_m, lr, beta1, beta2, eps, state);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_argmax_hits(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                       const uint8_t* mask, int32_t* pred, int32_t* hits, int* n_blocks_out) {
  const int blocks = ce_blocks(n);
  *n_blocks_out = blocks;
  if (n == 0) return 0;
  argmax_hits_rows<<<blocks, kCeWarps * 32, 0, (cudaStream_t)stream>>>(n, c, logits, ld, y, mask, pred, hits);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_normalize(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const int32_t* deg,
                     float* val) {
  if (n_rows == 0) return 0;
  normalize_rows<<<(unsigned)((n_rows + 7) / 8), 256, 0, (cudaStream_t)stream>>>(n_rows, rowptr, col, deg, val);
  note_launch();
  return (int)cudaGetLastError();
}

// dinv[i] = 1 / sqrt(deg[i]): the diagonal of D^-1/2 (degrees of A + I, so deg >= 1)
__global__ void inv_sqrt_degree(int64_t n, const int32_t* __restrict__ deg, float* __restrict__ dinv) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dinv[i] = 1.0f / sqrtf((float)deg[i]);
}
int launch_inv_sqrt_degree(void* stream, int64_t n, const int32_t* deg, float* dinv) {
  if (n == 0) return 0;
  inv_sqrt_degree<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(n, deg, dinv);
  note_launch();
  return (int)cudaGetLastError();
}

// dst[i, :] = scale[i] * src[i, :] over nvec float4 per row (dst may be src)
__global__ void scale_rows(int64_t n, int nvec, const float* __restrict__ scale, const float4* src, int64_t lds4,
                           float4* dst, int64_t ldd4) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * nvec) return;
  const int64_t i = idx / nvec;
  const int j = (int)(idx - i * nvec);
  const float sc = __ldg(scale + i);
  float4 v = src[i * lds4 + j];
  v.x *= sc; v.y *= sc; v.z *= sc; v.w *= sc;
  dst[i * ldd4 + j] = v;
}
int launch_scale_rows(void* stream, int64_t n, int32_t f, const float* scale, const float* src, int64_t lds, float* dst,
                      int64_t ldd) {
  if (n == 0 || f == 0) return 0;
  const int nvec = (f + 3) / 4;
  const int64_t total = n * nvec;
  scale_rows<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      n, nvec, scale, reinterpret_cast<const float4*>(src), lds / 4, reinterpret_cast<float4*>(dst), ldd / 4);
  note_launch();
  return (int)cudaGetLastError();
}

__global__ void repitch_rows(int64_t n, int f, const float* __restrict__ src, float* __restrict__ dst, int64_t ld) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * f) return;
  const int64_t i = idx / f, j = idx - i * f;
  dst[i * ld + j] = src[idx];
}

int launch_repitch(void* stream, int64_t n, int32_t f, const float* src, float* dst, int64_t ld) {
  if (n == 0 || f == 0) return 0;
  const int64_t total = n * f;
  repitch_rows<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(n, f, src, dst, ld);
  note_launch();
  return (int)cudaGetLastError();
}

int launch_mean(void* stream, const float* src, int count, float* dst) {
  mean_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(src, count, dst);
  note_launch();
  return (int)cudaGetLastError();
}

}  // namespace gcnsa

namespace gcnsa {
// ---------------------------------------------------------------------------
// Column sums without any allocation.  The block partials live in a file-scope
// device array that every GPU loading this library holds until the process
// exits: GCNSA_COLSUM_STATIC_MAX_F columns x 592 block slots x 4 bytes = 2.3 MiB.
namespace {

constexpr int kStaticMaxF = GCNSA_COLSUM_STATIC_MAX_F;
constexpr int kStaticBlocks = 592;  // block slots of the array; colsum_blocks() uses at most 296 of them
static __device__ __align__(256) float g_colsum_scratch[(size_t)kStaticBlocks * kStaticMaxF];

// In host code the name g_colsum_scratch is only a stand-in for the symbol, not
// an address a kernel could use: the device address is looked up once per
// device, with that device current, and cached here.
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_ptr[kMaxDevices] = {nullptr};

}  // namespace

}  // namespace gcnsa

extern "C" int gcnsa_op_colsum_static(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out,
                                      int32_t accumulate) {
  using namespace gcnsa;
  if (n < 0 || f < 0) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (f > kStaticMaxF)
    return fail(GCNSA_ERR_TOO_LARGE, "gcnsa_op_colsum_static: f exceeds GCNSA_COLSUM_STATIC_MAX_F columns; use "
                                     "gcnsa_op_colsum with caller-provided scratch");
  if (f == 0) return GCNSA_OK;
  if (!out || (n > 0 && !g) || ldg < f) return fail(GCNSA_ERR_ARG, "NULL pointer or leading dimension too small");
  if (colsum_scratch(n, f) > sizeof(float) * (size_t)kStaticBlocks * kStaticMaxF)
    return fail(GCNSA_ERR_TOO_LARGE, "gcnsa_op_colsum_static: built-in scratch too small");
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(GCNSA_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(GCNSA_ERR_ARG, "device index beyond the supported range");
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {  // first call on this device: resolve the symbol (no allocation takes place)
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_colsum_scratch);
      if (e != cudaSuccess) return fail(GCNSA_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
      g_static_ptr[dev] = (float*)p;
    }
    scratch = g_static_ptr[dev];
  }
  // every partial the second kernel reads is written by the first one in this
  // call, so nothing left behind by an earlier call needs clearing
  int rc = launch_colsum(stream, n, f, g, ldg, out, accumulate, scratch);
  if (rc != 0) return fail(GCNSA_ERR_CUDA, std::string("colsum launch: ") + cudaGetErrorString((cudaError_t)rc));
  return GCNSA_OK;
}

