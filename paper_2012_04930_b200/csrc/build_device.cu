// gcnsa_build_partitions on the device: the master's one-time step of Section 3.2
// in CUDA kernels.  The graph is uploaded once; then, for every partition p,
//   - Algorithm 1 (Section 3.1) runs as breadth-first levels toward all other
//     partitions at once: a sweep over p's cut edges marks level 1, every level
//     is counted per other partition, and each partition whose level holds at
//     least the vertices still wanted takes the ones with the smallest 64-bit
//     selection keys (a most-significant-byte-first radix select; keys never
//     tie, so the selected set does not depend on thread order), the others
//     take the whole level and expand it inside their own partition;
//   - the graph induced on owned + sampled vertices (Section 4: all other edges
//     are dropped) is written row by row, owned neighbours first, then sampled
//     ones, the self-loop merged in, which is ascending local order;
//   - the transposed CSR comes from a stable radix sort of (column, row) pairs,
//     a real transpose that assumes nothing about symmetry;
//   - rows are ordered hub rows first, then by descending length class (stable
//     radix sort), the loss rows and the transposed CSR over loss columns are
//     compacted in order.
// All integer work; results are bit-identical to the host builder's.  No kernel
// waits on another: every loop is bounded by a row length, a tile or 8 digits.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <string>
#include <vector>

#include "internal.h"
#include "parts.h"

namespace gcnsa {

namespace {

constexpr unsigned kFull = 0xffffffffu;
typedef unsigned long long u64;

#if GCNSA_DBG
GCNSA_DBG_WORD(g_dbg_build);
// a position a kernel is about to write must lie inside the range it was given
#define GCNSA_CHECK_WRITE(pos, limit, code) dbg_in(&g_dbg_build, (pos), 0, (limit), (code))
#else
#define GCNSA_CHECK_WRITE(pos, limit, code) true
#endif

__host__ __device__ inline uint64_t mix64d(uint64_t z) {  // SplitMix64 finalizer (Steele, Lea, Flood 2014)
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
// state of the selection key after the seed and the four stream words; the key of vertex v is mix64d(state ^ v)
__host__ __device__ inline uint64_t key_state(uint64_t seed, uint64_t w0, uint64_t w1, uint64_t w2, uint64_t w3) {
  uint64_t h = mix64d(seed);
  h = mix64d(h ^ w0);
  h = mix64d(h ^ w1);
  h = mix64d(h ^ w2);
  return mix64d(h ^ w3);
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline unsigned blocks_for(int64_t items, int per_block) { return (unsigned)std::max<int64_t>(1, ceil_div(items, per_block)); }
__device__ inline int64_t global_thread() { return (int64_t)blockIdx.x * blockDim.x + threadIdx.x; }
__device__ inline int64_t global_warp() { return global_thread() >> 5; }
__device__ inline int lane_id() { return threadIdx.x & 31; }

// ------------------------------------------------------------------ scan ---
constexpr int kScanThreads = 512, kScanItems = 8, kScanTile = kScanThreads * kScanItems;

__global__ void __launch_bounds__(kScanThreads) scan_tile_sums(const int32_t* __restrict__ in, int64_t n, int64_t* tile_sum) {
  __shared__ int64_t ws[kScanThreads / 32];
  const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
  int64_t s = 0;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k)
    if (base + k < n) s += in[base + k];
  for (int off = 16; off; off >>= 1) s += __shfl_down_sync(kFull, s, off);
  if (lane_id() == 0) ws[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    int64_t t = threadIdx.x < kScanThreads / 32 ? ws[threadIdx.x] : 0;
    for (int off = 16; off; off >>= 1) t += __shfl_down_sync(kFull, t, off);
    if (threadIdx.x == 0) tile_sum[blockIdx.x] = t;
  }
}

// inclusive scan of one value per thread over a block of NT threads; *total = the block's sum
template <int NT>
__device__ inline int64_t block_inclusive_scan(int64_t v, int64_t* ws /* [NT / 32] shared */, int64_t* total) {
  const int lane = lane_id(), warp = threadIdx.x >> 5;
  int64_t x = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int64_t y = __shfl_up_sync(kFull, x, off);
    if (lane >= off) x += y;
  }
  if (lane == 31) ws[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int64_t w = lane < NT / 32 ? ws[lane] : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int64_t y = __shfl_up_sync(kFull, w, off);
      if (lane >= off) w += y;
    }
    if (lane < NT / 32) ws[lane] = w;
  }
  __syncthreads();
  const int64_t r = x + (warp ? ws[warp - 1] : 0);
  *total = ws[NT / 32 - 1];
  __syncthreads();  // ws may be reused by the caller
  return r;
}

// one block: tile_sum[0 .. nt) becomes its exclusive scan, tile_sum[nt] the total
__global__ void __launch_bounds__(1024) scan_tile_offsets(int64_t* tile_sum, int64_t nt) {
  __shared__ int64_t ws[32];
  int64_t carry = 0;
  for (int64_t base = 0; base < nt; base += 1024) {
    const int64_t i = base + threadIdx.x;
    const int64_t v = i < nt ? tile_sum[i] : 0;
    int64_t total;
    const int64_t incl = block_inclusive_scan<1024>(v, ws, &total);
    if (i < nt) tile_sum[i] = carry + incl - v;
    carry += total;
  }
  if (threadIdx.x == 0) tile_sum[nt] = carry;
}

template <class OutT>
__global__ void __launch_bounds__(kScanThreads) scan_apply(const int32_t* in, int64_t n, const int64_t* __restrict__ tile_off,
                                                           OutT* out) {
  __shared__ int64_t ws[kScanThreads / 32];
  const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
  int32_t v[kScanItems];
  int64_t s = 0;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    v[k] = base + k < n ? in[base + k] : 0;
    s += v[k];
  }
  int64_t total;
  const int64_t incl = block_inclusive_scan<kScanThreads>(s, ws, &total);
  int64_t run = tile_off[blockIdx.x] + incl - s;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    if (base + k < n) out[base + k] = (OutT)run;
    run += v[k];
  }
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) out[n] = (OutT)tile_off[gridDim.x];
}

// ---------------------------------------------------------- input checks ---
// err holds the smallest (position * 8 + code id) seen; ~0 = none
constexpr int kErrArg = 1, kErrLoopDup = 2, kErrNotSym = 3, kErrLabel = 4;
__device__ inline void report(u64* err, int64_t pos, int id) { atomicMin(err, (u64)pos * 8 + (u64)id); }

__global__ void check_rowptr(const int64_t* __restrict__ rp, int64_t n, int64_t nnz, u64* err) {
  const int64_t v = global_thread();
  if (v >= n) return;
  if (rp[v] < 0 || rp[v + 1] < rp[v] || rp[v + 1] > nnz) report(err, v, kErrArg);
}

__global__ void check_rows(const int64_t* __restrict__ rp, const int32_t* __restrict__ col, int64_t n, u64* err) {
  const int64_t v = global_warp();
  if (v >= n) return;
  const int64_t b = rp[v], e1 = rp[v + 1];
  for (int64_t e = b + lane_id(); e < e1; e += 32) {
    const int64_t u = col[e];
    if (u < 0 || u >= n) { report(err, e, kErrArg); continue; }
    if (u == v) report(err, e, kErrLoopDup);
    if (e > b) {
      const int64_t prev = col[e - 1];
      if (prev == u) report(err, e, kErrLoopDup);
      else if (prev > u) report(err, e, kErrArg);
    }
  }
}

__global__ void check_symmetry(const int64_t* __restrict__ rp, const int32_t* __restrict__ col, int64_t n, u64* err) {
  const int64_t v = global_warp();
  if (v >= n) return;
  const int64_t b = rp[v], e1 = rp[v + 1];
  for (int64_t e = b + lane_id(); e < e1; e += 32) {
    const int64_t u = col[e];
    int64_t lo = rp[u], hi = rp[u + 1];  // v must be in the ascending row of u
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      if (col[mid] < v) lo = mid + 1;
      else hi = mid;
    }
    if (lo >= rp[u + 1] || col[lo] != v) report(err, e, kErrNotSym);
  }
}

__global__ void check_range_i32(const int32_t* __restrict__ a, int64_t n, int32_t limit, u64* err) {
  const int64_t v = global_thread();
  if (v < n && (a[v] < 0 || a[v] >= limit)) report(err, v, kErrLabel);
}

// ------------------------------------------------------------ assignment ---
__global__ void assign_range(int32_t* part, int64_t n, int64_t m) {
  const int64_t v = global_thread();
  if (v < n) part[v] = (int32_t)((v * m) / n);
}

// ------------------------------------------- batched radix select (64-bit) ---
// Select s looks for the key with exactly sel_rank[s] smaller keys among its candidates.  One pass per byte,
// most significant first: a histogram of the byte among the candidates that agree with the bytes already
// fixed, then select_decide fixes the next byte.  After 8 passes sel_prefix[s] is that key.
__global__ void select_decide(u64* sel_prefix, int64_t* sel_rank, const int32_t* __restrict__ sel_on, unsigned* hist,
                              int shift) {
  __shared__ int64_t ws[8];
  const int s = blockIdx.x, t = threadIdx.x;  // 256 threads: one per bin
  const unsigned c = hist[(size_t)s * 256 + t];
  hist[(size_t)s * 256 + t] = 0;  // ready for the next pass
  int64_t total;
  const int64_t incl = block_inclusive_scan<256>((int64_t)c, ws, &total);
  if (!sel_on[s]) return;
  const int64_t excl = incl - c, r = sel_rank[s];
  __syncthreads();  // every thread has read the rank before one of them rewrites it
  if (c > 0 && excl <= r && r < incl) {
    sel_prefix[s] |= (u64)t << shift;
    sel_rank[s] = r - excl;
  }
}

// candidates of select q: every vertex (hash assignment: the key at each cut rank of the ordering)
__global__ void select_hist_all(int64_t n, int n_sel, uint64_t state, const u64* __restrict__ sel_prefix, unsigned* hist,
                                int shift) {
  const int64_t v = global_thread();
  if (v >= n) return;
  const uint64_t key = mix64d(state ^ (uint64_t)v);
  for (int s = 0; s < n_sel; ++s) {
    if (shift < 56 && (key >> (shift + 8)) != (sel_prefix[s] >> (shift + 8))) continue;
    atomicAdd(&hist[(size_t)s * 256 + ((key >> shift) & 255)], 1u);
  }
}

__global__ void assign_from_cuts(int32_t* part, int64_t n, int n_sel, uint64_t state, const u64* __restrict__ cut_key) {
  const int64_t v = global_thread();
  if (v >= n) return;
  const uint64_t key = mix64d(state ^ (uint64_t)v);
  int q = 0;
  for (int s = 0; s < n_sel; ++s) q += key >= cut_key[s];  // cut keys ascend; a repeated rank repeats its key
  part[v] = q;
}

// --------------------------------------------------------- Algorithm 1 ---
struct Alg1State {       // device arrays of m entries each
  int64_t* need;         // vertices still wanted from partition q
  int32_t* active;       // the walk toward q goes on
  int32_t* mode;         // this level: 0 nothing, 1 take the whole level and expand, 2 select by key
  u64* cnt;              // size of the current level inside q
  int32_t* depth;        // deepest level used
  uint64_t* hstate;      // key state of (p, q, level) for the selecting partitions
  u64* sel_prefix;
  int64_t* sel_rank;
  int32_t* sel_on;
  int32_t* flags;        // [0] some partition expands, [1] some partition selects
};

__global__ void count_owned(const int32_t* __restrict__ part, int64_t n, u64* cnt) {
  const int64_t v = global_thread();
  const int q = v < n ? part[v] : -1;
  const unsigned peers = __match_any_sync(kFull, q);
  if (q >= 0 && (peers & ((1u << lane_id()) - 1)) == 0) atomicAdd(&cnt[q], (u64)__popc(peers));
}

// level 1 toward every other partition: the vertices outside p adjacent to a vertex of p
__global__ void mark_level1(const int64_t* __restrict__ rp, const int32_t* __restrict__ col, const int32_t* __restrict__ part,
                            int64_t n, int32_t p, int32_t* mark) {
  const int64_t v = global_warp();
  if (v >= n || part[v] != p) return;
  for (int64_t e = rp[v] + lane_id(); e < rp[v + 1]; e += 32) {
    const int32_t u = col[e];
    if (part[u] != p) mark[u] = 1;
  }
}

__global__ void level_count(const int32_t* __restrict__ mark, const int32_t* __restrict__ part, int64_t n, int32_t level,
                            Alg1State st) {
  const int64_t v = global_thread();
  int q = -1;
  if (v < n && mark[v] == level && st.active[part[v]]) q = part[v];
  const unsigned peers = __match_any_sync(kFull, q);
  if (q >= 0 && (peers & ((1u << lane_id()) - 1)) == 0) atomicAdd(&st.cnt[q], (u64)__popc(peers));
}

// one block
__global__ void level_decide(int32_t m, int32_t p, int32_t level, uint64_t seed, Alg1State st) {
  if (threadIdx.x == 0) { st.flags[0] = 0; st.flags[1] = 0; }
  __syncthreads();
  for (int q = threadIdx.x; q < m; q += blockDim.x) {
    int mode = 0, on = 0;
    if (q != p && st.active[q]) {
      const int64_t c = (int64_t)st.cnt[q];
      if (c == 0) {
        st.active[q] = 0;  // nothing further is reachable: the sample toward q stays short
      } else {
        st.depth[q] = level;
        if (c >= st.need[q]) {
          mode = 2; on = 1;
          st.sel_rank[q] = st.need[q] - 1;
          st.sel_prefix[q] = 0;
          st.hstate[q] = key_state(seed, 2, (uint64_t)p, (uint64_t)q, (uint64_t)level);
          st.need[q] = 0;
          st.active[q] = 0;
          st.flags[1] = 1;
        } else {
          mode = 1;
          st.need[q] -= c;
          st.flags[0] = 1;
        }
      }
    }
    st.mode[q] = mode;
    st.sel_on[q] = on;
    st.cnt[q] = 0;
  }
}

__global__ void select_hist_level(const int32_t* __restrict__ mark, const int32_t* __restrict__ part, int64_t n, int32_t level,
                                  Alg1State st, unsigned* hist, int shift) {
  const int64_t v = global_thread();
  if (v >= n || mark[v] != level) return;
  const int q = part[v];
  if (st.mode[q] != 2) return;
  const uint64_t key = mix64d(st.hstate[q] ^ (uint64_t)v);
  if (shift < 56 && (key >> (shift + 8)) != (st.sel_prefix[q] >> (shift + 8))) return;
  atomicAdd(&hist[(size_t)q * 256 + ((key >> shift) & 255)], 1u);
}

__global__ void take_selected(const int32_t* __restrict__ mark, const int32_t* __restrict__ part, int64_t n, int32_t level,
                              Alg1State st, int32_t* taken) {
  const int64_t v = global_thread();
  if (v >= n || mark[v] != level) return;
  const int q = part[v];
  if (st.mode[q] == 2 && mix64d(st.hstate[q] ^ (uint64_t)v) <= st.sel_prefix[q]) taken[v] = 1;
}

// partitions in mode 1: the whole level is taken and its unvisited neighbours inside the same partition form
// the next level (several writers store the same level number)
__global__ void take_and_expand(const int64_t* __restrict__ rp, const int32_t* __restrict__ col,
                                const int32_t* __restrict__ part, int64_t n, int32_t level, Alg1State st, int32_t* mark,
                                int32_t* taken) {
  const int64_t v = global_warp();
  if (v >= n || mark[v] != level) return;
  const int q = part[v];
  if (st.mode[q] != 1) return;
  if (lane_id() == 0) taken[v] = 1;
  for (int64_t e = rp[v] + lane_id(); e < rp[v + 1]; e += 32) {
    const int32_t w = col[e];
    if (part[w] == q && mark[w] == 0) mark[w] = level + 1;
  }
}

// ----------------------------------------------------- lists and rows ---
__global__ void flag_equal(const int32_t* __restrict__ a, int64_t n, int32_t value, int32_t* flag) {
  const int64_t i = global_thread();
  if (i < n) flag[i] = a[i] == value;
}

// out[offset + pos[i]] = src ? src[i] : i for the flagged i (pos = exclusive scan of flag)
__global__ void scatter_flagged(const int32_t* __restrict__ flag, const int32_t* __restrict__ pos, int64_t n,
                                const int32_t* __restrict__ src, int32_t* out, int64_t offset) {
  const int64_t i = global_thread();
  if (i < n && flag[i]) out[offset + pos[i]] = src ? src[i] : (int32_t)i;
}

__global__ void set_g2l(const int32_t* __restrict__ members, int64_t np, int32_t* g2l) {
  const int64_t i = global_thread();
  if (i < np) g2l[members[i]] = (int32_t)i;
}

__device__ inline int warp_sum(int x) {
  for (int off = 16; off; off >>= 1) x += __shfl_xor_sync(kFull, x, off);
  return x;
}

// deg[i] = 1 + neighbours of members[i] inside the extended partition
__global__ void induced_count(const int64_t* __restrict__ rp, const int32_t* __restrict__ col,
                              const int32_t* __restrict__ members, int64_t np, const int32_t* __restrict__ g2l, int32_t* deg) {
  const int64_t i = global_warp();
  if (i >= np) return;
  const int64_t v = members[i];
  int c = 0;
  for (int64_t e = rp[v] + lane_id(); e < rp[v + 1]; e += 32) c += g2l[col[e]] >= 0;
  c = warp_sum(c);
  if (lane_id() == 0) deg[i] = c + 1;
}

// row i: [owned neighbours ascending] ++ [sampled neighbours ascending], self-loop merged in.  Owned vertices
// have the local ids below n_owned in ascending global order and so have the sampled ones above, hence the row
// is ascending in local ids.
__global__ void induced_fill(const int64_t* __restrict__ rp, const int32_t* __restrict__ col,
                             const int32_t* __restrict__ members, int64_t np, int64_t n_owned,
                             const int32_t* __restrict__ g2l, const int32_t* __restrict__ rowptr, int32_t* out) {
  const int64_t i = global_warp();
  if (i >= np) return;
  const int64_t v = members[i];
  const int lane = lane_id();
  const unsigned lt = (1u << lane) - 1;
  int32_t* w = out + rowptr[i];
  const int len = rowptr[i + 1] - rowptr[i];  // read by the checks of the debug build only
  (void)len;
  int base = 0, below = 0;  // kept so far; kept with a local id below i
  const int64_t b = rp[v], e1 = rp[v + 1];
  for (int pass = 0; pass < 2; ++pass) {
    for (int64_t e0 = b; e0 < e1; e0 += 32) {
      const int64_t e = e0 + lane;
      int32_t l = -1;
      if (e < e1) l = g2l[col[e]];
      const bool keep = l >= 0 && ((l < n_owned) == (pass == 0));
      const unsigned kept = __ballot_sync(kFull, keep);
      const unsigned less = __ballot_sync(kFull, keep && l < (int32_t)i);
      if (keep) {
        const int at = base + __popc(kept & lt) + (l > (int32_t)i ? 1 : 0);
        if (GCNSA_CHECK_WRITE(at, len, kDbgInducedWrite)) w[at] = l;
      }
      base += __popc(kept);
      below += __popc(less);
    }
  }
  if (lane == 0 && GCNSA_CHECK_WRITE(below, len, kDbgInducedWrite)) w[below] = (int32_t)i;
}

__global__ void expand_rows(const int32_t* __restrict__ rowptr, int64_t np, int32_t* rowid) {
  const int64_t i = global_warp();
  if (i >= np) return;
  for (int32_t e = rowptr[i] + lane_id(); e < rowptr[i + 1]; e += 32) rowid[e] = (int32_t)i;
}

__global__ void count_columns(const int32_t* __restrict__ col, int64_t nnz, int32_t* cnt) {
  const int64_t e = global_thread();
  if (e < nnz) atomicAdd(&cnt[col[e]], 1);
}

// key[i] = order_key of row i (hub rows, then the others window by window, by descending length class), val[i] = i
__global__ void length_keys(const int32_t* __restrict__ rowptr, int64_t np, int64_t thr, int64_t window, uint32_t* key,
                            int32_t* val) {
  const int64_t i = global_thread();
  if (i < np) {
    key[i] = order_key(rowptr[i + 1] - rowptr[i], thr, np, i, window);
    val[i] = (int32_t)i;
  }
}

// out[0] += rows of at least thr entries; with carries: only rows that carry loss, and out[1] += their entries
__global__ void count_long_rows(const int32_t* __restrict__ rowptr, int64_t np, int64_t thr,
                                const uint8_t* __restrict__ carries, u64* out) {
  const int64_t i = global_thread();
  int is_long = 0, len = 0;
  if (i < np && (!carries || carries[i])) {
    len = rowptr[i + 1] - rowptr[i];
    is_long = len >= thr;
  }
  const unsigned any_long = __ballot_sync(kFull, is_long);
  const int total = warp_sum(carries ? len : 0);
  if (lane_id() == 0) {
    if (any_long) atomicAdd(&out[0], (u64)__popc(any_long));
    if (carries && total) atomicAdd(&out[1], (u64)total);
  }
}

// labels, loss mask and (as int32 flags) who carries loss, in partition order
__global__ void gather_labels(const int32_t* __restrict__ members, int64_t np, int64_t lim, const int32_t* __restrict__ y,
                              const uint8_t* __restrict__ train_mask, int32_t* y_out, uint8_t* mask_out) {
  const int64_t i = global_thread();
  if (i >= np) return;
  const int32_t v = members[i];
  y_out[i] = y[v];
  mask_out[i] = (i < lim && train_mask[v] != 0) ? 1 : 0;
}

__global__ void flag_carrying_in_order(const int32_t* __restrict__ order, int64_t np, const uint8_t* __restrict__ carries,
                                       int32_t* flag) {
  const int64_t k = global_thread();
  if (k < np) flag[k] = carries[order[k]];
}

__global__ void restricted_count(const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col, int64_t np,
                                 const uint8_t* __restrict__ carries, int32_t* cnt) {
  const int64_t j = global_warp();
  if (j >= np) return;
  int c = 0;
  for (int32_t e = t_rowptr[j] + lane_id(); e < t_rowptr[j + 1]; e += 32) c += carries[t_col[e]];
  c = warp_sum(c);
  if (lane_id() == 0) cnt[j] = c;
}

__global__ void restricted_fill(const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col, int64_t np,
                                const uint8_t* __restrict__ carries, const int32_t* __restrict__ tm_rowptr, int32_t* out) {
  const int64_t j = global_warp();
  if (j >= np) return;
  const int lane = lane_id();
  const unsigned lt = (1u << lane) - 1;
  int32_t* w = out + tm_rowptr[j];
  const int len = tm_rowptr[j + 1] - tm_rowptr[j];  // read by the checks of the debug build only
  (void)len;
  int base = 0;
  const int32_t b = t_rowptr[j], e1 = t_rowptr[j + 1];
  for (int32_t e0 = b; e0 < e1; e0 += 32) {
    const int32_t e = e0 + lane;
    int32_t r = -1;
    if (e < e1) r = t_col[e];
    const bool keep = r >= 0 && carries[r];
    const unsigned kept = __ballot_sync(kFull, keep);
    if (keep) {
      const int at = base + __popc(kept & lt);
      if (GCNSA_CHECK_WRITE(at, len, kDbgLossColWrite)) w[at] = r;
    }
    base += __popc(kept);
  }
}

// x_out[i, :] = x[members[i], :], pad columns zero
__global__ void gather_features(const float* __restrict__ x, int64_t f, const int32_t* __restrict__ members, int64_t np,
                                float* x_out, int64_t ld) {
  const int64_t i = global_warp();
  if (i >= np) return;
  const float* src = x + (int64_t)members[i] * f;
  float* dst = x_out + i * ld;
  for (int64_t c = lane_id(); c < ld; c += 32) dst[c] = c < f ? src[c] : 0.f;
}

// ------------------------------------------- stable radix sort (32-bit keys) ---
// Least significant byte first.  A block owns a tile of kSortTile consecutive elements and each of its warps
// a contiguous slice of that tile.  Pass = per-tile byte histogram, one scan over [byte][tile], then a scatter
// in which every warp walks its slice in order and ranks equal bytes by lane (match_any), so equal keys keep
// their input order.
constexpr int kSortWarps = 8, kSortRounds = 8, kSortSlice = 32 * kSortRounds, kSortTile = kSortWarps * kSortSlice;

__global__ void __launch_bounds__(kSortWarps * 32) sort_hist(const uint32_t* __restrict__ key, int64_t n, int shift,
                                                             int32_t* hist, int64_t n_tiles) {
  __shared__ int cnt[256];
  cnt[threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kSortTile;
  for (int r = 0; r < kSortRounds; ++r) {
    const int64_t i = base + (int64_t)r * (kSortWarps * 32) + threadIdx.x;
    if (i < n) atomicAdd(&cnt[(key[i] >> shift) & 255], 1);
  }
  __syncthreads();
  hist[(int64_t)threadIdx.x * n_tiles + blockIdx.x] = cnt[threadIdx.x];
}

__global__ void __launch_bounds__(kSortWarps * 32) sort_scatter(const uint32_t* __restrict__ key, const int32_t* __restrict__ val,
                                                                int64_t n, int shift, const int32_t* __restrict__ offset,
                                                                int64_t n_tiles, uint32_t* key_out, int32_t* val_out) {
  __shared__ int wc[kSortWarps][256];
  const int warp = threadIdx.x >> 5, lane = lane_id();
  for (int w = 0; w < kSortWarps; ++w) wc[w][threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * kSortSlice;
  for (int r = 0; r < kSortRounds; ++r) {
    const int64_t i = base + r * 32 + lane;
    if (i < n) atomicAdd(&wc[warp][(key[i] >> shift) & 255], 1);
  }
  __syncthreads();
  {  // thread d: where each warp's elements with byte d start
    const int d = threadIdx.x;
    int run = offset[(int64_t)d * n_tiles + blockIdx.x];
    for (int w = 0; w < kSortWarps; ++w) {
      const int c = wc[w][d];
      wc[w][d] = run;
      run += c;
    }
  }
  __syncthreads();
  for (int r = 0; r < kSortRounds; ++r) {
    const int64_t i = base + r * 32 + lane;
    const bool valid = i < n;
    uint32_t k = 0;
    int d = 256;  // lanes past the end form a group of their own
    if (valid) {
      k = key[i];
      d = (k >> shift) & 255;
    }
    const unsigned peers = __match_any_sync(kFull, d);
    const int rank = __popc(peers & ((1u << lane) - 1));
    int pos = 0;
    if (valid) pos = wc[warp][d] + rank;
    __syncwarp();
    if (valid) {
      if (GCNSA_CHECK_WRITE(pos, n, kDbgSortWrite)) {
        key_out[pos] = k;
        val_out[pos] = val[i];
      }
      if (rank == 0) wc[warp][d] += __popc(peers);
    }
    __syncwarp();
  }
}

// -------------------------------------------------------------- host side ---
struct Builder {
  gcnsa_parts* P;
  const gcnsa_graph* g;
  const gcnsa_part_opts* o;
  cudaStream_t s;
  std::vector<void*> tmp;  // scratch, released when the build ends
  int rc = GCNSA_OK;

  // whole graph on the device
  int64_t* rp = nullptr;
  int32_t* col = nullptr;
  float* x = nullptr;
  int32_t* y = nullptr;
  uint8_t* train_mask = nullptr;
  int32_t* part = nullptr;
  // per-vertex scratch
  int32_t *mark = nullptr, *taken = nullptr, *g2l = nullptr, *flag = nullptr, *pos = nullptr;
  int64_t* tiles = nullptr;  // scan scratch
  int64_t tiles_cap = 0;
  u64* err = nullptr;
  u64* counters = nullptr;   // 8 words
  unsigned* sel_hist = nullptr;
  Alg1State st{};
  // pinned-free host mirror for small reads
  u64 h_words[8];

  ~Builder() {
    cudaStreamSynchronize(s);
    for (void* p : tmp) P->env.release(p);
  }
  bool ok() const { return rc == GCNSA_OK; }
  int cuda(cudaError_t e, const char* what) {
    if (e != cudaSuccess && ok()) rc = fail(GCNSA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
    return rc;
  }
  int launched(const char* what) {
    note_launch();
    return cuda(cudaGetLastError(), what);
  }
  template <class T>
  T* scratch(size_t count) {
    if (!ok()) return nullptr;
    void* p = P->env.alloc(std::max<size_t>(count, 1) * sizeof(T));
    if (!p) { rc = fail(GCNSA_ERR_OOM, "device allocation failed (partition build scratch)"); return nullptr; }
    tmp.push_back(p);
    return (T*)p;
  }
  void drop(void* p) {  // early release of a scratch buffer (stream-ordered allocators reuse it safely after a sync)
    if (!p) return;
    auto it = std::find(tmp.begin(), tmp.end(), p);
    if (it != tmp.end()) {
      cudaStreamSynchronize(s);
      P->env.release(p);
      tmp.erase(it);
    }
  }
  template <class T>
  T* result(size_t count) {
    if (!ok()) return nullptr;
    void* p = P->dalloc(std::max<size_t>(count, 1) * sizeof(T));
    if (!p) { rc = fail(GCNSA_ERR_OOM, "device allocation failed"); return nullptr; }
    return (T*)p;
  }
  template <class T>
  T* upload(const T* host, size_t count) {
    T* d = scratch<T>(count);
    if (d && count) cuda(cudaMemcpyAsync(d, host, count * sizeof(T), cudaMemcpyHostToDevice, s), "upload");
    return d;
  }
  void zero(void* p, size_t bytes) {
    if (ok() && bytes) cuda(cudaMemsetAsync(p, 0, bytes, s), "cudaMemsetAsync");
  }
  void fill_ff(void* p, size_t bytes) {
    if (ok() && bytes) cuda(cudaMemsetAsync(p, 0xFF, bytes, s), "cudaMemsetAsync");
  }
  template <class T>
  void read(T* host, const void* dev, size_t count) {  // synchronizes
    if (!ok()) return;
    cuda(cudaMemcpyAsync(host, dev, count * sizeof(T), cudaMemcpyDeviceToHost, s), "download");
    cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");
  }

  // out[0 .. n] = exclusive scan of in[0 .. n); returns a device pointer to the int64 total
  template <class OutT>
  const int64_t* scan(const int32_t* in, int64_t n, OutT* out) {
    if (!ok()) return nullptr;
    const int64_t nt = std::max<int64_t>(1, ceil_div(n, kScanTile));
    if (nt + 1 > tiles_cap) { rc = fail(GCNSA_ERR_ARG, "internal: scan scratch too small"); return nullptr; }
    scan_tile_sums<<<(unsigned)nt, kScanThreads, 0, s>>>(in, n, tiles);
    launched("scan_tile_sums");
    scan_tile_offsets<<<1, 1024, 0, s>>>(tiles, nt);
    launched("scan_tile_offsets");
    scan_apply<OutT><<<(unsigned)nt, kScanThreads, 0, s>>>(in, n, tiles, out);
    launched("scan_apply");
    return tiles + nt;
  }
  int64_t scan_total(const int64_t* dev_total) {
    int64_t t = 0;
    read(&t, dev_total, 1);
    return t;
  }

  // stable sort of (key, val) by key over `bits` low bits; the result is in (k0, v0) or (k1, v1): returns which
  int sort_pairs(uint32_t* k0, int32_t* v0, uint32_t* k1, int32_t* v1, int64_t n, int bits, int32_t* hist) {
    int cur = 0;
    const int64_t n_tiles = std::max<int64_t>(1, ceil_div(n, kSortTile));
    for (int shift = 0; shift < bits && ok(); shift += 8) {
      const uint32_t* ki = cur ? k1 : k0;
      const int32_t* vi = cur ? v1 : v0;
      uint32_t* ko = cur ? k0 : k1;
      int32_t* vo = cur ? v0 : v1;
      sort_hist<<<(unsigned)n_tiles, kSortWarps * 32, 0, s>>>(ki, n, shift, hist, n_tiles);
      launched("sort_hist");
      scan<int32_t>(hist, 256 * n_tiles, hist);
      sort_scatter<<<(unsigned)n_tiles, kSortWarps * 32, 0, s>>>(ki, vi, n, shift, hist, n_tiles, ko, vo);
      launched("sort_scatter");
      cur ^= 1;
    }
    return cur;
  }

  // 8 passes of the batched radix select over n_sel selects (state already set up on the device)
  template <class HistLaunch>
  void select_passes(int n_sel, u64* sel_prefix, int64_t* sel_rank, const int32_t* sel_on, HistLaunch&& hist_launch) {
    for (int shift = 56; shift >= 0 && ok(); shift -= 8) {
      hist_launch(shift);
      launched("select_hist");
      select_decide<<<(unsigned)n_sel, 256, 0, s>>>(sel_prefix, sel_rank, sel_on, sel_hist, shift);
      launched("select_decide");
    }
  }

  int check_err_word() {  // reads the error word of the input checks
    u64 w = ~0ull;
    read(&w, err, 1);
    if (!ok() || w == ~0ull) return rc;
    switch ((int)(w & 7)) {
      case kErrLoopDup: return rc = fail(GCNSA_ERR_SELF_LOOP_OR_DUP, "graph rows must be without loops or repeats");
      case kErrNotSym: return rc = fail(GCNSA_ERR_NOT_SYMMETRIC, "edge (u,v) present without (v,u)");
      case kErrLabel: return rc = fail(GCNSA_ERR_LABEL_RANGE, "label or partition id out of range");
      default: return rc = fail(GCNSA_ERR_ARG, "graph rows must be in range and ascending");
    }
  }

  int run();
  void assign();
  void build_partition(int32_t p, int64_t n_owned);
};

void Builder::assign() {
  const int64_t n = g->n;
  const int32_t m = o->m;
  if (o->part_mode == GCNSA_PART_RANGE) {
    assign_range<<<blocks_for(n, 256), 256, 0, s>>>(part, n, m);
    launched("assign_range");
  } else if (o->part_mode == GCNSA_PART_USER) {
    cuda(cudaMemcpyAsync(part, o->user_part, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, s), "upload");
    cuda(cudaMemsetAsync(err, 0xFF, sizeof(u64), s), "cudaMemsetAsync");
    check_range_i32<<<blocks_for(n, 256), 256, 0, s>>>(part, n, m, err);
    launched("check_range_i32");
    if (check_err_word() == GCNSA_ERR_LABEL_RANGE) rc = fail(GCNSA_ERR_LABEL_RANGE, "user_part outside [0, m)");
  } else {
    // rank r of the key ordering goes to partition floor(r m / n): vertex v is in partition q iff its key is at
    // least the key of rank ceil(q n / m) for exactly q of the cuts q = 1 .. m - 1
    const int n_sel = m - 1;
    const uint64_t state = key_state(o->seed, 1, 0, 0, 0);
    if (n_sel > 0) {
      std::vector<int64_t> ranks((size_t)n_sel);
      std::vector<int32_t> on((size_t)n_sel, 1);
      for (int q = 1; q < m; ++q) ranks[q - 1] = (int64_t)(((__int128)q * n + m - 1) / m);
      cuda(cudaMemcpyAsync(st.sel_rank, ranks.data(), ranks.size() * sizeof(int64_t), cudaMemcpyHostToDevice, s), "upload");
      cuda(cudaMemcpyAsync(st.sel_on, on.data(), on.size() * sizeof(int32_t), cudaMemcpyHostToDevice, s), "upload");
      zero(st.sel_prefix, (size_t)n_sel * sizeof(u64));
      cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");  // the host vectors go out of scope
      select_passes(n_sel, st.sel_prefix, st.sel_rank, st.sel_on, [&](int shift) {
        select_hist_all<<<blocks_for(n, 256), 256, 0, s>>>(n, n_sel, state, st.sel_prefix, sel_hist, shift);
      });
    }
    assign_from_cuts<<<blocks_for(n, 256), 256, 0, s>>>(part, n, n_sel, state, st.sel_prefix);
    launched("assign_from_cuts");
  }
}

void Builder::build_partition(int32_t p, int64_t n_owned) {
  const int64_t n = g->n;
  const int32_t m = o->m;
  DevPart& d = P->parts[p];
  d.info = gcnsa_part_info{};
  d.info.n_owned = n_owned;
  const int64_t nts = m > 1 ? (int64_t)(((unsigned __int128)o->overlap_ppm * (unsigned __int128)n_owned) /
                                        ((unsigned __int128)1000000 * (unsigned __int128)(m - 1)))
                            : 0;
  d.info.nts = nts;
  d.depth.assign((size_t)m, 0);
  const unsigned vb = blocks_for(n, 256), wb = blocks_for(n * 32, 256);

  // ---- Algorithm 1 toward every other partition
  zero(taken, (size_t)n * sizeof(int32_t));
  if (nts > 0) {
    zero(mark, (size_t)n * sizeof(int32_t));
    std::vector<int64_t> need((size_t)m, nts);
    std::vector<int32_t> active((size_t)m, 1);
    need[p] = 0; active[p] = 0;
    cuda(cudaMemcpyAsync(st.need, need.data(), (size_t)m * sizeof(int64_t), cudaMemcpyHostToDevice, s), "upload");
    cuda(cudaMemcpyAsync(st.active, active.data(), (size_t)m * sizeof(int32_t), cudaMemcpyHostToDevice, s), "upload");
    zero(st.cnt, (size_t)m * sizeof(u64));
    zero(st.depth, (size_t)m * sizeof(int32_t));
    cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    mark_level1<<<wb, 256, 0, s>>>(rp, col, part, n, p, mark);
    launched("mark_level1");
    for (int64_t level = 1; level <= n && ok(); ++level) {
      level_count<<<vb, 256, 0, s>>>(mark, part, n, (int32_t)level, st);
      launched("level_count");
      level_decide<<<1, 256, 0, s>>>(m, p, (int32_t)level, o->seed, st);
      launched("level_decide");
      int32_t flags[2] = {0, 0};
      read(flags, st.flags, 2);
      if (!ok()) return;
      if (flags[1]) {
        select_passes(m, st.sel_prefix, st.sel_rank, st.sel_on, [&](int shift) {
          select_hist_level<<<vb, 256, 0, s>>>(mark, part, n, (int32_t)level, st, sel_hist, shift);
        });
        take_selected<<<vb, 256, 0, s>>>(mark, part, n, (int32_t)level, st, taken);
        launched("take_selected");
      }
      if (!flags[0]) break;
      take_and_expand<<<wb, 256, 0, s>>>(rp, col, part, n, (int32_t)level, st, mark, taken);
      launched("take_and_expand");
    }
    read(d.depth.data(), st.depth, (size_t)m);
    for (int32_t q = 0; q < m; ++q) d.info.max_depth = std::max(d.info.max_depth, d.depth[q]);
  }
  if (!ok()) return;

  // ---- members: owned ascending, then sampled ascending
  const int64_t* halo_total = scan<int32_t>(taken, n, pos);
  const int64_t n_halo = scan_total(halo_total);
  if (!ok()) return;
  const int64_t np = n_owned + n_halo;
  if (np >= (int64_t)INT32_MAX) { rc = fail(GCNSA_ERR_TOO_LARGE, "extended partition has 2^31 rows or more"); return; }
  d.info.n_halo = n_halo;
  d.info.n = np;
  P->n_max = std::max(P->n_max, np);
  int32_t* members = scratch<int32_t>((size_t)np);
  if (!ok()) return;
  scatter_flagged<<<vb, 256, 0, s>>>(taken, pos, n, nullptr, members, n_owned);
  launched("scatter_flagged");
  flag_equal<<<vb, 256, 0, s>>>(part, n, p, flag);
  launched("flag_equal");
  scan<int32_t>(flag, n, pos);
  scatter_flagged<<<vb, 256, 0, s>>>(flag, pos, n, nullptr, members, 0);
  launched("scatter_flagged");
  fill_ff(g2l, (size_t)n * sizeof(int32_t));
  const unsigned pvb = blocks_for(np, 256), pwb = blocks_for(np * 32, 256);
  set_g2l<<<pvb, 256, 0, s>>>(members, np, g2l);
  launched("set_g2l");

  // ---- induced rows + self-loops
  int32_t* deg = scratch<int32_t>((size_t)np + 1);
  d.rowptr = result<int32_t>((size_t)np + 1);
  if (!ok()) return;
  induced_count<<<pwb, 256, 0, s>>>(rp, col, members, np, g2l, deg);
  launched("induced_count");
  const int64_t nnz = scan_total(scan<int32_t>(deg, np, d.rowptr));
  if (!ok()) return;
  if (nnz >= (int64_t)INT32_MAX) { rc = fail(GCNSA_ERR_TOO_LARGE, "extended partition has 2^31 non-zeros or more"); return; }
  d.info.nnz = nnz;
  d.col = result<int32_t>((size_t)nnz);
  if (!ok()) return;
  induced_fill<<<pwb, 256, 0, s>>>(rp, col, members, np, n_owned, g2l, d.rowptr, d.col);
  launched("induced_fill");

  // ---- transpose: stable sort of (column, row) by column
  int bits = 1;
  while (((int64_t)1 << bits) <= np) ++bits;  // keys are in [0, np]
  const int64_t sort_tiles = std::max<int64_t>(1, ceil_div(nnz, kSortTile));
  uint32_t* k0 = scratch<uint32_t>((size_t)nnz);
  int32_t* v0 = scratch<int32_t>((size_t)nnz);
  uint32_t* k1 = scratch<uint32_t>((size_t)nnz);
  int32_t* v1 = scratch<int32_t>((size_t)nnz);
  int32_t* hist = scratch<int32_t>((size_t)(256 * sort_tiles + 1));
  int32_t* cnt = scratch<int32_t>((size_t)np + 1);
  d.t_rowptr = result<int32_t>((size_t)np + 1);
  d.t_col = result<int32_t>((size_t)nnz);
  if (!ok()) return;
  cuda(cudaMemcpyAsync(k0, d.col, (size_t)nnz * sizeof(int32_t), cudaMemcpyDeviceToDevice, s), "copy");
  expand_rows<<<pwb, 256, 0, s>>>(d.rowptr, np, v0);
  launched("expand_rows");
  zero(cnt, ((size_t)np + 1) * sizeof(int32_t));
  count_columns<<<blocks_for(nnz, 256), 256, 0, s>>>(d.col, nnz, cnt);
  launched("count_columns");
  scan<int32_t>(cnt, np, d.t_rowptr);
  {
    const int where = sort_pairs(k0, v0, k1, v1, nnz, bits, hist);
    cuda(cudaMemcpyAsync(d.t_col, where ? v1 : v0, (size_t)nnz * sizeof(int32_t), cudaMemcpyDeviceToDevice, s), "copy");
  }

  // ---- labels, loss mask
  const int64_t lim = o->loss_on_halo ? np : n_owned;
  d.y = result<int32_t>((size_t)np);
  d.mask = result<uint8_t>((size_t)np);
  if (!ok()) return;
  gather_labels<<<pvb, 256, 0, s>>>(members, np, lim, y, train_mask, d.y, d.mask);
  launched("gather_labels");

  // ---- processing orders (longest rows first, ties by row index) and hub-row counts
  d.order = result<int32_t>((size_t)np);
  d.t_order = result<int32_t>((size_t)np);
  d.tm_order = result<int32_t>((size_t)np);
  d.tm_rowptr = result<int32_t>((size_t)np + 1);
  if (!ok()) return;
  const int64_t window = order_window_rows(o->order_window, np);
  auto make_order = [&](const int32_t* rowptr, int64_t row_thr, int32_t* order_out) {
    length_keys<<<pvb, 256, 0, s>>>(rowptr, np, row_thr, window, k0, v0);
    launched("length_keys");
    const int where = sort_pairs(k0, v0, k1, v1, np, order_key_bits(np, window), hist);
    cuda(cudaMemcpyAsync(order_out, where ? v1 : v0, (size_t)np * sizeof(int32_t), cudaMemcpyDeviceToDevice, s), "copy");
  };
  const int64_t thr = long_row_threshold(nnz);
  make_order(d.rowptr, thr, d.order);
  make_order(d.t_rowptr, thr, d.t_order);
  zero(counters, 8 * sizeof(u64));
  count_long_rows<<<pvb, 256, 0, s>>>(d.rowptr, np, thr, nullptr, counters + 0);
  launched("count_long_rows");
  count_long_rows<<<pvb, 256, 0, s>>>(d.t_rowptr, np, thr, nullptr, counters + 2);
  launched("count_long_rows");
  count_long_rows<<<pvb, 256, 0, s>>>(d.rowptr, np, thr, d.mask, counters + 4);  // loss rows: [4] long ones, [5] entries
  launched("count_long_rows");

  // ---- the rows that carry loss, in processing order
  flag_carrying_in_order<<<pvb, 256, 0, s>>>(d.order, np, d.mask, flag);
  launched("flag_carrying_in_order");
  const int64_t n_train = scan_total(scan<int32_t>(flag, np, pos));
  if (!ok()) return;
  d.info.n_train = n_train;
  d.m_order = result<int32_t>((size_t)n_train);
  if (!ok()) return;
  scatter_flagged<<<pvb, 256, 0, s>>>(flag, pos, np, d.order, d.m_order, 0);
  launched("scatter_flagged");

  // ---- transposed CSR over the columns that carry loss
  restricted_count<<<pwb, 256, 0, s>>>(d.t_rowptr, d.t_col, np, d.mask, cnt);
  launched("restricted_count");
  const int64_t tm_nnz = scan_total(scan<int32_t>(cnt, np, d.tm_rowptr));
  if (!ok()) return;
  d.tm_nnz = tm_nnz;
  d.tm_col = result<int32_t>((size_t)tm_nnz);
  if (!ok()) return;
  restricted_fill<<<pwb, 256, 0, s>>>(d.t_rowptr, d.t_col, np, d.mask, d.tm_rowptr, d.tm_col);
  launched("restricted_fill");
  make_order(d.tm_rowptr, long_row_threshold(tm_nnz), d.tm_order);
  count_long_rows<<<pvb, 256, 0, s>>>(d.tm_rowptr, np, long_row_threshold(tm_nnz), nullptr, counters + 6);
  launched("count_long_rows");
  read(h_words, counters, 8);
  if (!ok()) return;
  d.n_long = (int64_t)h_words[0];
  d.t_n_long = (int64_t)h_words[2];
  d.m_n_long = (int64_t)h_words[4];
  d.m_nnz = (int64_t)h_words[5];
  d.tm_n_long = (int64_t)h_words[6];

  // the sort scratch is the largest: give it back before the values and features are allocated
  drop(k0); drop(v0); drop(k1); drop(v1); drop(hist);

  // ---- features in partition order
  d.x = result<float>((size_t)np * (size_t)P->ldx);
  if (!ok()) return;
  gather_features<<<pwb, 256, 0, s>>>(x, g->f, members, np, d.x, P->ldx);
  launched("gather_features");

  // ---- D^-1/2 (A + I) D^-1/2: entry (i, j) and entry (j, i) of the transpose are both 1 / sqrt(d_i d_j)
  d.val = result<float>((size_t)nnz);
  d.t_val = result<float>((size_t)nnz);
  d.tm_val = result<float>((size_t)tm_nnz);
  d.dinv = result<float>((size_t)np);
  if (!ok()) return;
  int e = launch_normalize(s, np, d.rowptr, d.col, deg, d.val);
  if (!e) e = launch_inv_sqrt_degree(s, np, deg, d.dinv);
  if (!e) e = launch_normalize(s, np, d.t_rowptr, d.t_col, deg, d.t_val);
  if (!e) e = launch_normalize(s, np, d.tm_rowptr, d.tm_col, deg, d.tm_val);
  if (e) { cuda((cudaError_t)e, "normalize"); return; }

  // ---- host copies of the small things
  std::vector<int32_t> mem32((size_t)np);
  read(mem32.data(), members, (size_t)np);
  if (!ok()) return;
  d.members.assign(mem32.begin(), mem32.end());
  drop(members); drop(deg); drop(cnt);
}

int Builder::run() {
  const int64_t n = g->n, nnz = g->nnz;
  const int32_t m = o->m;
  if (g->rowptr[0] != 0 || g->rowptr[n] != nnz) return fail(GCNSA_ERR_ARG, "rowptr[0] != 0 or rowptr[n] != nnz");
  const unsigned vb = blocks_for(n, 256), wb = blocks_for(n * 32, 256);

  // ---- the graph goes to the device once
  rp = upload(g->rowptr, (size_t)n + 1);
  col = upload(g->col, (size_t)nnz);
  y = upload(g->y, (size_t)n);
  train_mask = upload(g->train_mask, (size_t)n);
  err = scratch<u64>(1);
  counters = scratch<u64>(8);
  part = scratch<int32_t>((size_t)n);
  if (!ok()) return rc;

  // ---- input checks (each needs what the one before it established)
  fill_ff(err, sizeof(u64));
  check_rowptr<<<vb, 256, 0, s>>>(rp, n, nnz, err);
  launched("check_rowptr");
  if (check_err_word()) return rc;
  check_rows<<<wb, 256, 0, s>>>(rp, col, n, err);
  launched("check_rows");
  if (check_err_word()) return rc;
  check_symmetry<<<wb, 256, 0, s>>>(rp, col, n, err);
  launched("check_symmetry");
  check_range_i32<<<vb, 256, 0, s>>>(y, n, g->c, err);
  launched("check_range_i32");
  if (check_err_word()) {
    if (rc == GCNSA_ERR_LABEL_RANGE) rc = fail(rc, "label outside [0, c)");
    return rc;
  }

  // ---- scratch per vertex, state of the walks and of the selects
  const int64_t max_items = std::max<int64_t>(n, 1) + 1;
  mark = scratch<int32_t>((size_t)n);
  taken = scratch<int32_t>((size_t)n);
  g2l = scratch<int32_t>((size_t)n);
  flag = scratch<int32_t>((size_t)n);
  pos = scratch<int32_t>((size_t)n + 1);
  // scans run over per-vertex arrays and over the sort's [256][tiles] histograms (at most nnz_p / 8 + 256 entries)
  tiles_cap = ceil_div(std::max<int64_t>(max_items, (int64_t)INT32_MAX / 8 + 512), kScanTile) + 2;
  tiles = scratch<int64_t>((size_t)tiles_cap);
  const size_t ms = (size_t)std::max<int32_t>(m, 1);
  st.need = scratch<int64_t>(ms);
  st.active = scratch<int32_t>(ms);
  st.mode = scratch<int32_t>(ms);
  st.cnt = scratch<u64>(ms);
  st.depth = scratch<int32_t>(ms);
  st.hstate = scratch<uint64_t>(ms);
  st.sel_prefix = scratch<u64>(ms);
  st.sel_rank = scratch<int64_t>(ms);
  st.sel_on = scratch<int32_t>(ms);
  st.flags = scratch<int32_t>(2);
  sel_hist = scratch<unsigned>(ms * 256);
  if (!ok()) return rc;
  zero(sel_hist, ms * 256 * sizeof(unsigned));
  zero(st.mode, ms * sizeof(int32_t));

  // ---- assignment and partition sizes
  assign();
  if (!ok()) return rc;
  P->part.resize((size_t)n);
  u64* owned_cnt = scratch<u64>(ms);
  if (!ok()) return rc;
  zero(owned_cnt, ms * sizeof(u64));
  count_owned<<<vb, 256, 0, s>>>(part, n, owned_cnt);
  launched("count_owned");
  std::vector<u64> n_owned(ms, 0);
  read(n_owned.data(), owned_cnt, ms);
  read(P->part.data(), part, (size_t)n);
  if (!ok()) return rc;

  // ---- features: uploaded dense, gathered per partition on the device
  x = scratch<float>((size_t)n * (size_t)g->f);
  if (!ok()) return rc;
  cuda(cudaMemcpy2DAsync(x, (size_t)g->f * sizeof(float), g->x, (size_t)g->ldx * sizeof(float), (size_t)g->f * sizeof(float),
                         (size_t)n, cudaMemcpyHostToDevice, s),
       "upload of the features");

  for (int32_t p = 0; p < m && ok(); ++p) build_partition(p, (int64_t)n_owned[p]);
  if (ok()) cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");
  return rc;
}

}  // namespace

int build_device(gcnsa_parts* P, const gcnsa_graph* g, const gcnsa_part_opts* o) {
  Builder b{P, g, o, P->env.stream()};
  P->parts.assign((size_t)o->m, DevPart());
  P->n_max = 0;
  return b.run();
}

int debug_word_build(unsigned long long* out, bool clear) {
  *out = 0ull;
#if GCNSA_DBG
  cudaError_t e = cudaMemcpyFromSymbol(out, g_dbg_build, sizeof(*out));
  if (e == cudaSuccess && clear) {
    const unsigned long long zero = 0ull;
    e = cudaMemcpyToSymbol(g_dbg_build, &zero, sizeof(zero));
  }
  return (int)e;
#else
  (void)clear;
  return 0;
#endif
}

}  // namespace gcnsa
