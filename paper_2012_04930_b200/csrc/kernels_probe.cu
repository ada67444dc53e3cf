// A measuring stick for the sparse products of the GCN layer (Section 4.1), not a step of the method: the rate
// at which the SMs can gather 512-byte rows of a row-major fp32 matrix when nothing else is asked of them.  Every
// warp adds up rows (32 lanes x float4) whose indices it computes itself - no index loads, no dependent addresses -
// with 16 gathers in flight per warp, 24 warps per SM.  What the CSR kernel reaches on the same matrix is read against this.
#include <cuda_runtime.h>

#include "internal.h"

namespace gcnsa {

namespace {

constexpr int kProbeUnroll = 16;
constexpr int kProbeThreads = 256;
constexpr int kProbeBlocksPerSm = 12;  // three resident at a time (the 16 rows in flight take 64 registers), four rounds

// One pseudo-random draw (a linear congruential step and one xor-shift), the same on the host side of the test.
__device__ __forceinline__ uint32_t probe_next(uint32_t s) {
  s = s * 1664525u + 1013904223u;
  return s ^ (s >> 15);
}

// Gather k of a round goes to the block's window of `window_rows` rows when hit_every > 0 and k % hit_every == 0
// (a handful of rows that stay in L1), otherwise to any of the n_rows rows.
__global__ void __launch_bounds__(kProbeThreads, 3)
gather_probe(const float4* __restrict__ x, int64_t ldx4, uint32_t n_rows, uint32_t window_rows, int hit_every, int rounds,
             float4* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const uint32_t gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  uint32_t s = 0x9E3779B9u * (gw + 1u);
  const uint32_t base = (blockIdx.x * 977u) % (n_rows - window_rows + 1u);
  // which of a round's 16 gathers go to the window: decided once, a division per gather would bound the loop
  uint32_t near_mask = 0;
  for (int u = 0; u < kProbeUnroll; ++u)
    if (hit_every > 0 && (u % hit_every) == 0) near_mask |= 1u << u;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int it = 0; it < rounds; ++it) {
    float4 v[kProbeUnroll];
#pragma unroll
    for (int u = 0; u < kProbeUnroll; ++u) {
      s = probe_next(s);
      const bool near = (near_mask >> u) & 1u;
      const uint32_t r = (near ? base : 0u) + __umulhi(s, near ? window_rows : n_rows);
      v[u] = __ldg(x + (int64_t)r * ldx4 + lane);
    }
#pragma unroll
    for (int u = 0; u < kProbeUnroll; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
  }
  out[(int64_t)gw * 32 + lane] = acc;
}

}  // namespace

int gather_probe_warps(int sms) { return sms * kProbeBlocksPerSm * (kProbeThreads / 32); }

int launch_gather_probe(void* stream, const float* x, int64_t ldx, int64_t n_rows, int32_t window_rows, int32_t hit_every,
                        int32_t rounds, float* out, int sms) {
  gather_probe<<<sms * kProbeBlocksPerSm, kProbeThreads, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const float4*>(x), ldx / 4, (uint32_t)n_rows, (uint32_t)window_rows, hit_every, rounds,
      reinterpret_cast<float4*>(out));
  note_launch();
  return (int)cudaGetLastError();
}

}  // namespace gcnsa
