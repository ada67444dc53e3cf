// GraphSAGE with the mean aggregator on the extended partitions (Section 4.1,
// "Investigated GCNs"; training scheme of Section 3.2): per mini-batch
//   1. a fixed number of neighbours is sampled for every vertex the batch needs
//      (the r smallest 64-bit selection keys among the vertex's neighbours
//      inside its extended partition: a uniform draw without replacement that
//      depends on (seed, partition, epoch, layer, vertex) only),
//   2. every layer is h_v = sigma([h_v | mean of the sampled neighbours] W + b),
//      the concatenation form of the published mean aggregator: the rows
//      [self | mean] are assembled by one gather kernel and multiplied by the
//      stacked matrix [W_self ; W_neigh] on the tensor cores,
//   3. softmax cross-entropy over the batch, the chain rule backwards (the mean
//      over a vertex's samples hands each sample 1 / count of the gradient),
//      one Adam step on the worker's copy of the parameters.
// The batch is laid out in slots: rows [0, nb) are the batch's vertices, row
// nb + i r2 + s is the s-th sampled neighbour of vertex i (r2 = fan-out of the
// output layer).  A vertex that several batch vertices sampled gets several
// slots; its embedding is the same in each (the hidden layer's sample depends
// on the vertex only), so the result is that of the definition and the
// backward pass needs no scatter: every slot has exactly one reader.
// All shapes are known to the host (batch size, fan-outs), so no step waits for
// a device value.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "internal.h"
#include "parts.h"

namespace gcnsa {

namespace {

constexpr unsigned kFull = 0xffffffffu;
typedef unsigned long long u64;

// SplitMix64 finalizer (Steele, Lea, Flood 2014) and the selection key built from it: the words are absorbed one
// at a time, the vertex id last
__host__ __device__ inline u64 mix64s(u64 z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
__host__ __device__ inline u64 key_prefix(u64 seed, u64 w0, u64 w1, u64 w2, u64 w3) {
  u64 h = mix64s(seed);
  h = mix64s(h ^ w0);
  h = mix64s(h ^ w1);
  h = mix64s(h ^ w2);
  return mix64s(h ^ w3);
}
constexpr u64 kTagNeighbor = 3, kTagBatch = 4;

inline unsigned blocks_for(int64_t items, int per_block) {
  return (unsigned)std::max<int64_t>(1, (items + per_block - 1) / per_block);
}

// ---------------------------------------------------------------- batches ---
// keys[i] = key(seed; 4, p, epoch, 0; list[i])
__global__ void sage_keys(const int32_t* __restrict__ list, int64_t n, u64 prefix, u64* __restrict__ keys) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) keys[i] = mix64s(prefix ^ (u64)list[i]);
}
// order[rank of keys[i]] = list[i]; keys are distinct (the key is a bijection of the vertex id), so the ranks are a
// permutation.  Brute force over tiles of keys in shared memory: n^2 comparisons, a millisecond at n = 10^5.
__global__ void __launch_bounds__(256)
sage_rank(const int32_t* __restrict__ list, const u64* __restrict__ keys, int64_t n, int32_t* __restrict__ order) {
  __shared__ u64 tile[1024];
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const u64 mine = i < n ? keys[i] : 0ull;
  int64_t rank = 0;
  for (int64_t t0 = 0; t0 < n; t0 += 1024) {
    const int cnt = (int)min((int64_t)1024, n - t0);
    for (int k = threadIdx.x; k < cnt; k += 256) tile[k] = keys[t0 + k];
    __syncthreads();
    if (i < n)
      for (int k = 0; k < cnt; ++k) rank += tile[k] < mine;
    __syncthreads();
  }
  if (i < n) order[rank] = list[i];
}

// --------------------------------------------------------------- sampling ---
// One warp per vertex vs[j] (-1 = none): its neighbours are the columns of its row of A + I other than itself.
// At most r of them: all, ascending.  More: the r with the smallest keys mix(prefix_v ^ u) (keys are distinct), in
// key order; out row j is padded with -1.
//
// Selection, r <= kFastR: one pipelined pass over the row collects the neighbours whose key is at most a threshold T
// into the warp's shared-memory list; the keys are uniform 64-bit numbers, so T = 2.5 r / deg of the key range
// catches about 2.5 r of them.  Between r and kCand candidates: their ranks among themselves (all pairs) are their
// ranks in the row, and ranks below r are the sample.  Fewer than r or more than kCand (rare): T is doubled / halved
// until both sides are bracketed, then bisected, and the pass repeated; the result never depends on T.
// Larger r: r rounds of "smallest key above the last one taken".
constexpr int kSampleWarps = 8, kCand = 128, kFastR = 50;

__global__ void __launch_bounds__(kSampleWarps * 32)
sage_sample(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, const int32_t* __restrict__ vs,
            int64_t n_v, int r, u64 seed, u64 p, u64 epoch_layer, const int64_t* __restrict__ batch_state,
            int32_t* __restrict__ out, int32_t* __restrict__ cnt) {
  // recorded batches: the epoch is read from the batch state, epoch_layer then carries the layer only
  if (batch_state) epoch_layer += (u64)batch_state[1] * 256;
  __shared__ u64 cand_key[kSampleWarps][kCand];
  __shared__ int32_t cand_id[kSampleWarps][kCand];
  const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  if (j >= n_v) return;
  int32_t* row = out + j * r;
  const int v = vs[j];
  if (v < 0) {
    for (int s = lane; s < r; s += 32) row[s] = -1;
    if (lane == 0) cnt[j] = 0;
    return;
  }
  const int beg = rowptr[v], end = rowptr[v + 1];
  const int deg = end - beg - 1;  // the self-loop is stored exactly once
  if (deg <= r) {
    for (int e = beg + lane; e < end; e += 32) {
      const int u = col[e];
      if (u < v) row[e - beg] = u;
      else if (u > v) row[e - beg - 1] = u;
    }
    for (int s = max(deg, 0) + lane; s < r; s += 32) row[s] = -1;
    if (lane == 0) cnt[j] = max(deg, 0);
    return;
  }
  const u64 prefix = key_prefix(seed, kTagNeighbor, p, epoch_layer, (u64)v);
  if (r <= kFastR) {
    u64* ck = cand_key[wib];
    int32_t* ci = cand_id[wib];
    const double want = 2.5 * (double)r / (double)deg;
    u64 T = want >= 1.0 ? ~0ull : (u64)(want * 18446744073709551615.0);
    u64 lo = 0ull, hi = ~0ull;       // count(lo) < r (or nothing known), count(hi) > kCand (or nothing known)
    bool have_lo = false, have_hi = false;
    int n_c = 0;
    for (int attempt = 0; attempt < 200; ++attempt) {   // every retry shrinks [lo, hi]; 64 bisections always suffice
      n_c = 0;
      for (int e0 = beg; e0 < end; e0 += 128) {
        int us[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {   // four loads in flight before the first key is needed
          const int e = e0 + 32 * t + lane;
          us[t] = e < end ? __ldg(col + e) : v;
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int u = us[t];
          const u64 k = mix64s(prefix ^ (u64)u);
          const bool take = u != v && k <= T;
          const unsigned m = __ballot_sync(kFull, take);
          if (take) {
            const int at = n_c + __popc(m & ((1u << lane) - 1));
            if (at < kCand) { ck[at] = k; ci[at] = u; }
          }
          n_c += __popc(m);
        }
      }
      if (n_c >= r && n_c <= kCand) break;
      if (n_c < r) { lo = T; have_lo = true; } else { hi = T; have_hi = true; }
      if (have_lo && have_hi) T = lo + (hi - lo) / 2;
      else if (have_lo) T = T > (~0ull >> 1) ? ~0ull : T * 2 + 1;
      else T = T / 2;
    }
    __syncwarp();
    for (int i = lane; i < n_c; i += 32) {
      const u64 mine = ck[i];
      int rank = 0;
      for (int q = 0; q < n_c; ++q) rank += ck[q] < mine;
      if (rank < r) row[rank] = ci[i];
    }
    if (lane == 0) cnt[j] = r;
    return;
  }
  u64 last = 0ull;
  for (int s = 0; s < r; ++s) {
    u64 best = 0ull;
    int who = -1;
    for (int e = beg + lane; e < end; e += 32) {
      const int u = col[e];
      if (u == v) continue;
      const u64 k = mix64s(prefix ^ (u64)u);
      if ((s == 0 || k > last) && (who < 0 || k < best)) { best = k; who = u; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const u64 ob = __shfl_xor_sync(kFull, best, off);
      const int ow = __shfl_xor_sync(kFull, who, off);
      if (ow >= 0 && (who < 0 || ob < best)) { best = ob; who = ow; }
    }
    if (lane == 0) row[s] = who;
    last = best;
  }
  if (lane == 0) cnt[j] = r;
}

// ------------------------------------------------------ [self | mean] rows ---
// out[j] = [ src[self_j] | mean over the samples of row j of src[.] ], both halves ld floats wide (f of them
// meaningful, the rest zero).  self_idx == NULL: self_j = j.  samp == NULL: the samples of row j are the rows
// slot_base + j r + s, s < cnt[j] (the slot layout of the batch).  A row without a vertex (self_j < 0) is zero.
__global__ void __launch_bounds__(256)
sage_concat_mean(const float* __restrict__ src, int64_t ld_src, int f, const int32_t* __restrict__ self_idx,
                 const int32_t* __restrict__ samp, const int32_t* __restrict__ cnt, int r, int64_t slot_base,
                 int64_t n_rows, float* __restrict__ out, int64_t ld) {
  const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (j >= n_rows) return;
  const int nvec = (f + 3) / 4, lvec = (int)(ld / 4);
  float4* o_self = reinterpret_cast<float4*>(out + j * 2 * ld);
  float4* o_mean = o_self + lvec;
  const int64_t self = self_idx ? (int64_t)self_idx[j] : j;
  const int c = self < 0 ? 0 : cnt[j];
  const float inv = c > 0 ? 1.0f / (float)c : 0.f;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int q0 = 0; q0 < lvec; q0 += 32) {
    const int q = q0 + lane;
    if (q >= lvec) break;
    float4 a = zero, m = zero;
    if (q < nvec && self >= 0) {
      a = __ldg(reinterpret_cast<const float4*>(src + self * ld_src) + q);
      for (int s = 0; s < c; ++s) {
        const int64_t u = samp ? (int64_t)__ldg(samp + j * r + s) : slot_base + j * r + s;
        const float4 t = __ldg(reinterpret_cast<const float4*>(src + u * ld_src) + q);
        m.x += t.x; m.y += t.y; m.z += t.z; m.w += t.w;
      }
      m.x *= inv; m.y *= inv; m.z *= inv; m.w *= inv;
    }
    o_self[q] = a;
    o_mean[q] = m;
  }
}

__global__ void sage_gather_labels(const int32_t* __restrict__ y, const int32_t* __restrict__ targets, int64_t nb,
                                   int32_t* __restrict__ yb) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < nb) yb[i] = y[targets[i]];
}

// Gradient w.r.t. the hidden layer's pre-activation, slot by slot.  dcat = G W^T has the layout of the [self | mean]
// rows: columns [0, ldh) belong to the batch vertex's own embedding, columns [ldh, 2 ldh) to the mean over its
// samples, of which each sample receives 1 / count.  ReLU'(z) = [h > 0].
__global__ void sage_hidden_grad(const float* __restrict__ dcat, const float* __restrict__ h1, const int32_t* __restrict__ cnt2,
                                 int64_t nb, int r2, int64_t ldh, int64_t n_rows, float* __restrict__ dz1) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_rows * ldh) return;
  const int64_t j = idx / ldh, c = idx - j * ldh;
  float g = 0.f;
  if (j < nb) {
    g = dcat[j * 2 * ldh + c];
  } else {
    const int64_t i = (j - nb) / r2, s = (j - nb) - i * r2;
    const int k = cnt2[i];
    if (s < k) g = dcat[i * 2 * ldh + ldh + c] / (float)k;
  }
  dz1[idx] = h1[idx] > 0.f ? g : 0.f;
}

// out[0] += number of source rows the [self | mean] kernel reads for these rows: 1 + cnt per row that has a vertex
__global__ void sage_count_reads(const int32_t* __restrict__ self_idx, const int32_t* __restrict__ cnt, int64_t n_rows,
                                 u64* out) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int c = 0;
  if (j < n_rows && (!self_idx || self_idx[j] >= 0)) c = 1 + cnt[j];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) c += __shfl_xor_sync(kFull, c, off);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(out, (u64)c);
}

// acc[0] += loss * weight (one thread): the running sum of the batch losses of a partition
// Batch state of the recorded batches: [0] = index of the batch in flight, [1] = epoch.  A replayed graph cannot
// take new kernel arguments, so the batch's first kernel advances the index itself and copies the batch's targets.
__global__ void sage_set_state(int64_t* state, int64_t b, int64_t epoch) {
  state[0] = b;
  state[1] = epoch;
}
// one block: every thread reads the old index before thread 0 writes the new one
__global__ void sage_begin_batch(int64_t* state, const int32_t* __restrict__ order, int batch, int32_t* __restrict__ targets) {
  const int64_t b = state[0] + 1;
  __syncthreads();
  for (int i = threadIdx.x; i < batch; i += blockDim.x) targets[i] = order[b * batch + i];
  if (threadIdx.x == 0) state[0] = b;
}

__global__ void sage_loss_add(float* acc, const float* loss, float weight) {
  if (threadIdx.x == 0 && blockIdx.x == 0) acc[0] += loss[0] * weight;
}
// epoch[0] += part[0] * scale; part[0] = 0
__global__ void sage_loss_fold(float* epoch, float* part, float scale) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    epoch[0] += part[0] * scale;
    part[0] = 0.f;
  }
}
// acc = (first ? 0 : acc) + w * scale
__global__ void sage_param_mean(int64_t count, const float* __restrict__ w, float* __restrict__ acc, int first, float scale) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) acc[i] = (first ? 0.f : acc[i]) + w[i] * scale;
}

}  // namespace
}  // namespace gcnsa

using namespace gcnsa;

struct gcnsa_sage {
  Env env;
  gcnsa_sage_opts o{};
  int32_t m = 0;
  int64_t f = 0, h = 0, c = 0, ldf = 0, ldh = 0, ldc = 0;
  int64_t count = 0, w1_off = 0, b1_off = 0, w2_off = 0, b2_off = 0;  // flat parameter layout
  int64_t max_rows1 = 0;  // batch (1 + r2): rows of the hidden layer per batch
  int64_t epoch = 0;
  // parameters: aggregated, the worker's working copy, the running mean, the batch gradient, moments per worker
  float *theta = nullptr, *work = nullptr, *acc = nullptr, *grad = nullptr, *am = nullptr, *av = nullptr;
  double* adam_state = nullptr;  // [m x 4]
  // batch order of one (partition, epoch)
  u64* keys = nullptr;
  int32_t* order = nullptr;
  int32_t order_p = -1;
  int64_t order_epoch = -1;
  uint64_t order_uid = 0;
  // the batch
  int32_t *b1 = nullptr, *cnt2 = nullptr, *s1 = nullptr, *cnt1 = nullptr, *yb = nullptr;
  uint8_t* ones = nullptr;
  float *cat1 = nullptr, *h1 = nullptr, *cat2 = nullptr, *logits = nullptr, *g = nullptr, *dcat2 = nullptr, *dz1 = nullptr;
  float* loss = nullptr;  // [0] batch loss, [1] partition sum, [2] epoch loss
  void *ws = nullptr, *sc = nullptr;
  size_t ws_bytes = 0;
  int64_t last_nb = 0, last_rows1 = 0;
  // recorded full-size batch of every worker (batch_graph): keyed by the partitions object
  int64_t* batch_state = nullptr;
  std::vector<cudaGraphExec_t> batch_exec;
  std::vector<int> batch_kernels;
  uint64_t batch_uid = 0;
  bool graph_off = false;
  // optional timing with CUDA events: classes 0 = [self | mean] gathers, 1 = dense products, 2 = everything else
  struct Rec { int cat; double bytes, flops; int64_t launches; };
  bool prof_on = false;
  std::vector<cudaEvent_t> ev;
  std::vector<Rec> recs;
  int64_t launches_mark = 0;
  u64* read_rows = nullptr;  // device: [0] source rows read by the hidden layer's gathers, [1] by the output layer's
  void prof_begin() {
    if (!prof_on) return;
    const size_t i = recs.size() * 2;
    while (ev.size() < i + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { prof_on = false; return; }
      ev.push_back(e);
    }
    launches_mark = gcnsa_launch_count();
    cudaEventRecord(ev[i], env.stream());
  }
  void prof_end(int cat, double bytes, double flops) {
    if (!prof_on) return;
    cudaEventRecord(ev[recs.size() * 2 + 1], env.stream());
    recs.push_back({cat, bytes, flops, gcnsa_launch_count() - launches_mark});
  }
  std::vector<void*> owned;
  void* dalloc(size_t bytes) {
    void* p = env.alloc(bytes);
    if (p) owned.push_back(p);
    return p;
  }
};

namespace {

int cuda_err(cudaError_t e, const char* what) { return fail(GCNSA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e)); }
#define SCK(call)                                        \
  do {                                                   \
    cudaError_t e_ = (call);                             \
    if (e_ != cudaSuccess) return cuda_err(e_, #call);   \
  } while (0)
#define SCKL(call)                                               \
  do {                                                           \
    int e_ = (call);                                             \
    if (e_ != 0) return cuda_err((cudaError_t)e_, #call);        \
  } while (0)
#define SLAUNCHED(what)                                          \
  do {                                                           \
    note_launch();                                               \
    cudaError_t e_ = cudaGetLastError();                         \
    if (e_ != cudaSuccess) return cuda_err(e_, what);            \
  } while (0)

int check_model(const gcnsa_sage* S, const gcnsa_parts* P) {
  if (!S || !P) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (P->m != S->m || P->f != S->f || P->c != S->c) return fail(GCNSA_ERR_ARG, "model was created for other partitions");
  return GCNSA_OK;
}

// the batch order of (p, epoch): the loss-carrying vertices of the partition in ascending key order
int ensure_order(gcnsa_sage* S, const gcnsa_parts* P, int32_t p, int64_t epoch) {
  if (S->order_p == p && S->order_epoch == epoch && S->order_uid == P->uid) return GCNSA_OK;
  const DevPart& d = P->parts[p];
  const int64_t nt = d.info.n_train;
  cudaStream_t s = S->env.stream();
  if (nt > 0) {
    const u64 prefix = key_prefix(S->o.seed, kTagBatch, (u64)p, (u64)epoch, 0);
    sage_keys<<<blocks_for(nt, 256), 256, 0, s>>>(d.m_order, nt, prefix, S->keys);
    SLAUNCHED("sage_keys");
    sage_rank<<<blocks_for(nt, 256), 256, 0, s>>>(d.m_order, S->keys, nt, S->order);
    SLAUNCHED("sage_rank");
  }
  S->order_p = p; S->order_epoch = epoch; S->order_uid = P->uid;
  return GCNSA_OK;
}

int64_t n_batches(const gcnsa_sage* S, const gcnsa_parts* P, int32_t p) {
  return (P->parts[p].info.n_train + S->o.batch - 1) / S->o.batch;
}

// recorded = true: the launches are being captured for replay; the batch index and the epoch then come from
// S->batch_state on the device (a full-size batch), b and epoch are not used
int run_batch(gcnsa_sage* S, const gcnsa_parts* P, int32_t p, int64_t epoch, int64_t b, bool apply, bool recorded = false) {
  int rc = recorded ? GCNSA_OK : ensure_order(S, P, p, epoch);
  if (rc) return rc;
  const DevPart& d = P->parts[p];
  cudaStream_t s = S->env.stream();
  void* sv = S->env.e.stream;
  const int64_t nt = d.info.n_train, B = S->o.batch;
  const int64_t nb = recorded ? B : std::min<int64_t>(B, nt - b * B);
  const int r1 = S->o.fanout[0], r2 = S->o.fanout[1];
  const int64_t rows1 = nb * (1 + r2);
  const int32_t* targets = S->order + b * B;
  const int mode = S->o.gemm_mode;

  // ---- the batch's vertices and their samples
  S->prof_begin();
  const int64_t* state = recorded ? S->batch_state : nullptr;
  const u64 ep = recorded ? 0 : (u64)epoch * 256;
  if (recorded) {
    sage_begin_batch<<<1, 256, 0, s>>>(S->batch_state, S->order, (int)B, S->b1);
    SLAUNCHED("sage_begin_batch");
  } else {
    SCK(cudaMemcpyAsync(S->b1, targets, (size_t)nb * sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
  }
  if (r2 > 0) {
    sage_sample<<<blocks_for(nb * 32, kSampleWarps * 32), kSampleWarps * 32, 0, s>>>(d.rowptr, d.col, S->b1, nb, r2, S->o.seed, (u64)p,
                                                        ep + 2, state, S->b1 + nb, S->cnt2);
    SLAUNCHED("sage_sample");
  } else {
    SCK(cudaMemsetAsync(S->cnt2, 0, (size_t)nb * sizeof(int32_t), s));
  }
  if (r1 > 0) {
    sage_sample<<<blocks_for(rows1 * 32, kSampleWarps * 32), kSampleWarps * 32, 0, s>>>(d.rowptr, d.col, S->b1, rows1, r1, S->o.seed, (u64)p,
                                                           ep + 1, state, S->s1, S->cnt1);
    SLAUNCHED("sage_sample");
  } else {
    SCK(cudaMemsetAsync(S->cnt1, 0, (size_t)rows1 * sizeof(int32_t), s));
  }
  if (S->prof_on) {
    sage_count_reads<<<blocks_for(rows1, 256), 256, 0, s>>>(S->b1, S->cnt1, rows1, S->read_rows);
    SLAUNCHED("sage_count_reads");
    sage_count_reads<<<blocks_for(nb, 256), 256, 0, s>>>(nullptr, S->cnt2, nb, S->read_rows + 1);
    SLAUNCHED("sage_count_reads");
  }
  S->prof_end(2, 0.0, 0.0);
  // ---- hidden layer: H1 = relu([x_v | mean x_u] [W_self ; W_neigh] + b)
  S->prof_begin();
  sage_concat_mean<<<blocks_for(rows1 * 32, 256), 256, 0, s>>>(d.x, P->ldx, (int)S->f, S->b1, S->s1, S->cnt1, r1, 0, rows1,
                                                              S->cat1, S->ldf);
  SLAUNCHED("sage_concat_mean");
  S->prof_end(0, 8.0 * (double)rows1 * (double)S->ldf, 0.0);  // the rows written; the rows read are counted on the device
  float* w = S->work;
  const double fl1 = 2.0 * (double)rows1 * (double)S->h * 2.0 * (double)S->f, fl2 = 2.0 * (double)nb * (double)S->c * 2.0 * (double)S->h;
  S->prof_begin();
  SCKL(launch_gemm(sv, mode, 0, 0, rows1, S->h, 2 * S->ldf, S->cat1, 2 * S->ldf, w + S->w1_off, S->ldh, S->h1, S->ldh, 0,
                   GCNSA_EPI_BIAS_RELU, w + S->b1_off, 0, S->ws, S->ws_bytes));
  S->prof_end(1, 0.0, fl1);
  // ---- output layer: logits = [h_v | mean h_u] [W_self ; W_neigh] + b, the samples of vertex i in slots nb + i r2 + s
  S->prof_begin();
  sage_concat_mean<<<blocks_for(nb * 32, 256), 256, 0, s>>>(S->h1, S->ldh, (int)S->h, nullptr, nullptr, S->cnt2, r2, nb, nb,
                                                           S->cat2, S->ldh);
  SLAUNCHED("sage_concat_mean");
  S->prof_end(0, 8.0 * (double)nb * (double)S->ldh, 0.0);
  S->prof_begin();
  SCKL(launch_gemm(sv, mode, 0, 0, nb, S->c, 2 * S->ldh, S->cat2, 2 * S->ldh, w + S->w2_off, S->ldc, S->logits, S->ldc, 0,
                   GCNSA_EPI_BIAS, w + S->b2_off, 0, S->ws, S->ws_bytes));
  S->prof_end(1, 0.0, fl2);
  // ---- loss over the batch and its gradient
  S->prof_begin();
  sage_gather_labels<<<blocks_for(nb, 256), 256, 0, s>>>(d.y, S->b1, nb, S->yb);
  SLAUNCHED("sage_gather_labels");
  SCKL(launch_softmax_ce(sv, nb, (int32_t)S->c, S->logits, S->ldc, S->yb, S->ones, nb, S->loss, S->g, S->ldc, S->sc));
  sage_loss_add<<<1, 32, 0, s>>>(S->loss + 1, S->loss, (float)nb);
  SLAUNCHED("sage_loss_add");
  S->prof_end(2, 0.0, 0.0);
  // ---- backward
  float* gr = S->grad;
  S->prof_begin();
  SCKL(launch_gemm(sv, mode, 1, 0, 2 * S->ldh, S->c, nb, S->cat2, 2 * S->ldh, S->g, S->ldc, gr + S->w2_off, S->ldc, 0,
                   GCNSA_EPI_NONE, nullptr, 0, S->ws, S->ws_bytes));
  SCKL(launch_gemm(sv, mode, 0, 1, nb, 2 * S->ldh, S->c, S->g, S->ldc, w + S->w2_off, S->ldc, S->dcat2, 2 * S->ldh, 0,
                   GCNSA_EPI_NONE, nullptr, 0, S->ws, S->ws_bytes));
  S->prof_end(1, 0.0, 2.0 * fl2);
  S->prof_begin();
  SCKL(launch_colsum(sv, nb, (int32_t)S->c, S->g, S->ldc, gr + S->b2_off, 0, S->sc));
  sage_hidden_grad<<<blocks_for(rows1 * S->ldh, 256), 256, 0, s>>>(S->dcat2, S->h1, S->cnt2, nb, std::max(r2, 1), S->ldh, rows1,
                                                                  S->dz1);
  SLAUNCHED("sage_hidden_grad");
  S->prof_end(2, 0.0, 0.0);
  S->prof_begin();
  SCKL(launch_gemm(sv, mode, 1, 0, 2 * S->ldf, S->h, rows1, S->cat1, 2 * S->ldf, S->dz1, S->ldh, gr + S->w1_off, S->ldh, 0,
                   GCNSA_EPI_NONE, nullptr, 0, S->ws, S->ws_bytes));
  S->prof_end(1, 0.0, fl1);
  S->prof_begin();
  SCKL(launch_colsum(sv, rows1, (int32_t)S->h, S->dz1, S->ldh, gr + S->b1_off, 0, S->sc));
  // ---- the worker's Adam step (its own moments and step count)
  if (apply) {
    double* st = S->adam_state + 4 * (size_t)p;
    SCKL(launch_adam_advance(sv, st, S->o.beta1, S->o.beta2));
    SCKL(launch_adam_dev(sv, S->count, S->work, S->grad, S->am + (size_t)p * S->count, S->av + (size_t)p * S->count, 1.0f,
                         S->o.lr, S->o.beta1, S->o.beta2, S->o.eps, st));
  }
  S->prof_end(2, 0.0, 0.0);
  S->last_nb = nb;
  S->last_rows1 = rows1;
  return GCNSA_OK;
}

}  // namespace

extern "C" {

int gcnsa_sage_destroy(gcnsa_sage* S) {
  if (!S) return GCNSA_OK;
  cudaStreamSynchronize(S->env.stream());
  for (void* p : S->owned) S->env.release(p);
  for (cudaEvent_t e : S->ev) cudaEventDestroy(e);
  for (cudaGraphExec_t g : S->batch_exec)
    if (g) cudaGraphExecDestroy(g);
  delete S;
  return GCNSA_OK;
}

int gcnsa_sage_create(const gcnsa_env* env, const gcnsa_parts* parts, const gcnsa_sage_opts* opts,
                      const float* const* w_self0, const float* const* w_neigh0, const float* const* b0, gcnsa_sage** out) {
  if (!out) return fail(GCNSA_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (!env || !parts || !opts || !w_self0 || !w_neigh0) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (opts->dims[0] != parts->f || opts->dims[2] != parts->c || opts->dims[1] < 1)
    return fail(GCNSA_ERR_ARG, "dims[0] must equal f, dims[2] must equal c of the partitions, dims[1] >= 1");
  if (opts->fanout[0] < 0 || opts->fanout[1] < 0 || opts->fanout[0] > 4096 || opts->fanout[1] > 4096 || opts->batch < 1 ||
      opts->batch > 65536)
    return fail(GCNSA_ERR_ARG, "fan-outs must be in [0, 4096] and the batch size in [1, 65536]");
  if (opts->gemm_mode != GCNSA_GEMM_FP32 && opts->gemm_mode != GCNSA_GEMM_TF32X3 && opts->gemm_mode != GCNSA_GEMM_TF32) return fail(GCNSA_ERR_ARG, "unknown gemm_mode");
  if (!(opts->lr > 0.f) || !(opts->beta1 >= 0.f && opts->beta1 < 1.f) || !(opts->beta2 >= 0.f && opts->beta2 < 1.f) ||
      !(opts->eps > 0.f))
    return fail(GCNSA_ERR_ARG, "Adam hyper-parameters out of range");
  for (int l = 0; l < 2; ++l)
    if (!w_self0[l] || !w_neigh0[l]) return fail(GCNSA_ERR_ARG, "w_self0[l] or w_neigh0[l] is NULL");
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count == 0) {
    cudaGetLastError();
    return fail(GCNSA_ERR_CUDA, "no CUDA device: this library has no CPU fallback");
  }
  gcnsa_sage* S = new (std::nothrow) gcnsa_sage();
  if (!S) return fail(GCNSA_ERR_OOM, "host allocation failed");
  S->env.e = *env;
  S->o = *opts;
  S->m = parts->m;
  S->f = opts->dims[0]; S->h = opts->dims[1]; S->c = opts->dims[2];
  S->ldf = GCNSA_LD(S->f); S->ldh = GCNSA_LD(S->h); S->ldc = GCNSA_LD(S->c);
  auto up64 = [](int64_t v) { return (v + 63) / 64 * 64; };
  int64_t off = 0;
  S->w1_off = off; off += up64(2 * S->ldf * S->ldh);
  S->b1_off = off; off += up64(S->ldh);
  S->w2_off = off; off += up64(2 * S->ldh * S->ldc);
  S->b2_off = off; off += up64(S->ldc);
  S->count = off;
  const int64_t B = opts->batch, r1 = opts->fanout[0], r2 = opts->fanout[1];
  S->max_rows1 = B * (1 + r2);
  int64_t nt_max = 1;
  for (int32_t p = 0; p < parts->m; ++p) nt_max = std::max<int64_t>(nt_max, parts->parts[p].info.n_train);
  auto fail_free = [&](int code) {
    const std::string keep = gcnsa_last_error();
    gcnsa_sage_destroy(S);
    return fail(code, keep);
  };
  const size_t pb = (size_t)S->count * sizeof(float);
  struct Want { void** slot; size_t bytes; };
  size_t ws = 0;
  const int mode = opts->gemm_mode;
  ws = std::max(ws, gemm_workspace(mode, 0, 0, S->max_rows1, S->h, 2 * S->ldf));
  ws = std::max(ws, gemm_workspace(mode, 0, 0, B, S->c, 2 * S->ldh));
  ws = std::max(ws, gemm_workspace(mode, 1, 0, 2 * S->ldh, S->c, B));
  ws = std::max(ws, gemm_workspace(mode, 0, 1, B, 2 * S->ldh, S->c));
  ws = std::max(ws, gemm_workspace(mode, 1, 0, 2 * S->ldf, S->h, S->max_rows1));
  // the last batch of a partition is smaller: its products have their own split along the inner dimension
  for (int64_t nb = 1; nb < B; ++nb) {
    ws = std::max(ws, gemm_workspace(mode, 0, 0, nb * (1 + r2), S->h, 2 * S->ldf));
    ws = std::max(ws, gemm_workspace(mode, 1, 0, 2 * S->ldf, S->h, nb * (1 + r2)));
    ws = std::max(ws, gemm_workspace(mode, 1, 0, 2 * S->ldh, S->c, nb));
    ws = std::max(ws, gemm_workspace(mode, 0, 1, nb, 2 * S->ldh, S->c));
    ws = std::max(ws, gemm_workspace(mode, 0, 0, nb, S->c, 2 * S->ldh));
  }
  S->ws_bytes = ws;
  const size_t sc = std::max(std::max(softmax_ce_scratch(B), colsum_scratch(S->max_rows1, (int32_t)S->h)),
                             colsum_scratch(B, (int32_t)S->c));
  const Want wants[] = {
      {(void**)&S->theta, pb}, {(void**)&S->work, pb}, {(void**)&S->acc, pb}, {(void**)&S->grad, pb},
      {(void**)&S->am, pb * (size_t)S->m}, {(void**)&S->av, pb * (size_t)S->m},
      {(void**)&S->adam_state, sizeof(double) * 4 * (size_t)S->m},
      {(void**)&S->keys, sizeof(u64) * (size_t)nt_max}, {(void**)&S->order, sizeof(int32_t) * (size_t)nt_max},
      {(void**)&S->b1, sizeof(int32_t) * (size_t)S->max_rows1}, {(void**)&S->cnt2, sizeof(int32_t) * (size_t)B},
      {(void**)&S->s1, sizeof(int32_t) * (size_t)(S->max_rows1 * std::max<int64_t>(r1, 1))},
      {(void**)&S->cnt1, sizeof(int32_t) * (size_t)S->max_rows1}, {(void**)&S->yb, sizeof(int32_t) * (size_t)B},
      {(void**)&S->ones, (size_t)B},
      {(void**)&S->cat1, sizeof(float) * (size_t)(S->max_rows1 * 2 * S->ldf)},
      {(void**)&S->h1, sizeof(float) * (size_t)(S->max_rows1 * S->ldh)},
      {(void**)&S->cat2, sizeof(float) * (size_t)(B * 2 * S->ldh)},
      {(void**)&S->logits, sizeof(float) * (size_t)(B * S->ldc)}, {(void**)&S->g, sizeof(float) * (size_t)(B * S->ldc)},
      {(void**)&S->dcat2, sizeof(float) * (size_t)(B * 2 * S->ldh)},
      {(void**)&S->dz1, sizeof(float) * (size_t)(S->max_rows1 * S->ldh)},
      {(void**)&S->loss, sizeof(float) * 4}, {(void**)&S->read_rows, sizeof(u64) * 2}, {(void**)&S->batch_state, sizeof(int64_t) * 2}, {&S->ws, ws}, {&S->sc, std::max<size_t>(sc, 256)}};
  cudaStream_t s = S->env.stream();
  for (const Want& wnt : wants) {
    *wnt.slot = S->dalloc(std::max<size_t>(wnt.bytes, 256));
    if (!*wnt.slot) {
      fail(GCNSA_ERR_OOM, "device allocation failed");
      return fail_free(GCNSA_ERR_OOM);
    }
    if (wnt.slot != &S->ws) {
      cudaError_t e = cudaMemsetAsync(*wnt.slot, 0, std::max<size_t>(wnt.bytes, 256), s);
      if (e != cudaSuccess) {
        cuda_err(e, "cudaMemsetAsync");
        return fail_free(GCNSA_ERR_CUDA);
      }
    }
  }
  cudaError_t e = cudaMemsetAsync(S->ones, 1, (size_t)B, s);
  // initial parameters: W_self in rows [0, f) of the stacked matrix, W_neigh in rows [ld, ld + f)
  const int64_t din[2] = {S->f, S->h}, dout[2] = {S->h, S->c}, ldin[2] = {S->ldf, S->ldh}, ldo[2] = {S->ldh, S->ldc};
  const int64_t w_off[2] = {S->w1_off, S->w2_off}, b_off[2] = {S->b1_off, S->b2_off};
  for (int l = 0; l < 2 && e == cudaSuccess; ++l) {
    float* wd = S->theta + w_off[l];
    const size_t hp = (size_t)dout[l] * sizeof(float), dp = (size_t)ldo[l] * sizeof(float);
    e = cudaMemcpy2DAsync(wd, dp, w_self0[l], hp, hp, (size_t)din[l], cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync(wd + ldin[l] * ldo[l], dp, w_neigh0[l], hp, hp, (size_t)din[l], cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && b0 && b0[l])
      e = cudaMemcpyAsync(S->theta + b_off[l], b0[l], hp, cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(S->work, S->theta, pb, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    cuda_err(e, "upload of the initial parameters");
    return fail_free(GCNSA_ERR_CUDA);
  }
  *out = S;
  return GCNSA_OK;
}

int gcnsa_sage_batches(const gcnsa_sage* S, const gcnsa_parts* P, int32_t p, int64_t* count_out) {
  int rc = check_model(S, P);
  if (rc) return rc;
  if (!count_out || p < 0 || p >= P->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  *count_out = n_batches(S, P, p);
  return GCNSA_OK;
}

int gcnsa_sage_batch(gcnsa_sage* S, const gcnsa_parts* P, int32_t p, int64_t epoch, int64_t b, int32_t apply,
                     float* loss_dev) {
  int rc = check_model(S, P);
  if (rc) return rc;
  if (p < 0 || p >= P->m || epoch < 0 || epoch >= (1LL << 40)) return fail(GCNSA_ERR_ARG, "partition index or epoch out of range");
  if (b < 0 || b >= n_batches(S, P, p)) return fail(GCNSA_ERR_ARG, "batch index out of range");
  rc = run_batch(S, P, p, epoch, b, apply != 0);
  if (rc) return rc;
  if (loss_dev) SCK(cudaMemcpyAsync(loss_dev, S->loss, sizeof(float), cudaMemcpyDeviceToDevice, S->env.stream()));
  return GCNSA_OK;
}

int gcnsa_sage_epoch(gcnsa_sage* S, const gcnsa_parts* P, float* loss_dev) {
  int rc = check_model(S, P);
  if (rc) return rc;
  cudaStream_t s = S->env.stream();
  const size_t pb = (size_t)S->count * sizeof(float);
  SCK(cudaMemsetAsync(S->loss, 0, 4 * sizeof(float), s));
  for (int32_t p = 0; p < P->m; ++p) {
    // the worker starts the epoch from the aggregated parameters (Section 3.2)
    SCK(cudaMemcpyAsync(S->work, S->theta, pb, cudaMemcpyDeviceToDevice, s));
    const int64_t nbatch = n_batches(S, P, p);
    int64_t b = 0;
    // the worker's full-size batches are one kernel sequence with the same shapes: recorded once per worker and
    // replayed, the batch index advancing on the device; the ragged last batch runs as plain launches
    const int64_t nfull = P->parts[p].info.n_train / S->o.batch;
    if (S->o.batch_graph && !S->graph_off && !S->prof_on && s != nullptr && nfull > 1) {
      rc = ensure_order(S, P, p, S->epoch);
      if (rc) return rc;
      if (S->batch_uid != P->uid || (int32_t)S->batch_exec.size() != P->m) {
        for (cudaGraphExec_t g : S->batch_exec)
          if (g) cudaGraphExecDestroy(g);
        S->batch_exec.assign((size_t)P->m, nullptr);
        S->batch_kernels.assign((size_t)P->m, 0);
        S->batch_uid = P->uid;
      }
      if (!S->batch_exec[p]) {
        const int64_t launches0 = gcnsa_launch_count();
        cudaGraph_t graph = nullptr;
        if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
          rc = run_batch(S, P, p, S->epoch, 0, true, true);
          const cudaError_t e = cudaStreamEndCapture(s, &graph);
          const int recorded = (int)(gcnsa_launch_count() - launches0);
          note_launch(-recorded);  // recorded, not launched
          if (rc != GCNSA_OK || e != cudaSuccess || !graph ||
              cudaGraphInstantiate(&S->batch_exec[p], graph, 0) != cudaSuccess) {
            S->batch_exec[p] = nullptr;
            S->graph_off = true;  // this stream or driver cannot record a batch: plain launches from now on
          }
          S->batch_kernels[p] = recorded;
          if (graph) cudaGraphDestroy(graph);
          cudaGetLastError();
        } else {
          cudaGetLastError();
          S->graph_off = true;
        }
      }
      if (S->batch_exec[p]) {
        sage_set_state<<<1, 1, 0, s>>>(S->batch_state, -1, S->epoch);
        SLAUNCHED("sage_set_state");
        for (; b < nfull; ++b) {
          SCK(cudaGraphLaunch(S->batch_exec[p], s));
          note_launch(S->batch_kernels[p]);
        }
        S->last_nb = S->o.batch;
        S->last_rows1 = (int64_t)S->o.batch * (1 + S->o.fanout[1]);
      }
    }
    for (; b < nbatch; ++b) {
      rc = run_batch(S, P, p, S->epoch, b, true);
      if (rc) return rc;
    }
    const int64_t nt = P->parts[p].info.n_train;
    sage_loss_fold<<<1, 32, 0, s>>>(S->loss + 2, S->loss + 1, nt > 0 ? 1.0f / ((float)nt * (float)P->m) : 0.f);
    SLAUNCHED("sage_loss_fold");
    sage_param_mean<<<blocks_for(S->count, 256), 256, 0, s>>>(S->count, S->work, S->acc, p == 0, 1.0f / (float)P->m);
    SLAUNCHED("sage_param_mean");
  }
  SCK(cudaMemcpyAsync(S->theta, S->acc, pb, cudaMemcpyDeviceToDevice, s));
  SCK(cudaMemcpyAsync(S->work, S->acc, pb, cudaMemcpyDeviceToDevice, s));
  if (loss_dev) SCK(cudaMemcpyAsync(loss_dev, S->loss + 2, sizeof(float), cudaMemcpyDeviceToDevice, s));
  S->epoch += 1;
  return GCNSA_OK;
}

int gcnsa_sage_profile(gcnsa_sage* S, int32_t enable) {
  if (!S) return fail(GCNSA_ERR_ARG, "model is NULL");
  SCK(cudaStreamSynchronize(S->env.stream()));
  S->prof_on = enable != 0;
  S->recs.clear();
  SCK(cudaMemsetAsync(S->read_rows, 0, 2 * sizeof(u64), S->env.stream()));
  return GCNSA_OK;
}

int gcnsa_sage_profile_read(gcnsa_sage* S, gcnsa_profile* out) {
  if (!S || !out) return fail(GCNSA_ERR_ARG, "NULL argument");
  std::memset(out, 0, sizeof(*out));
  SCK(cudaStreamSynchronize(S->env.stream()));
  for (size_t i = 0; i < S->recs.size(); ++i) {
    float ms = 0.f;
    SCK(cudaEventElapsedTime(&ms, S->ev[2 * i], S->ev[2 * i + 1]));
    const auto& r = S->recs[i];
    out->ms[r.cat] += ms;
    out->launches[r.cat] += r.launches;
    out->alg_bytes[r.cat] += r.bytes;
    out->flops[r.cat] += r.flops;
  }
  u64 rows[2] = {0, 0};
  SCK(cudaMemcpy(rows, S->read_rows, sizeof(rows), cudaMemcpyDeviceToHost));
  out->alg_bytes[0] += 4.0 * ((double)rows[0] * (double)S->f + (double)rows[1] * (double)S->h);
  for (int c = 0; c < 3; ++c) { out->l1_bytes[c] = out->alg_bytes[c]; out->alg_bytes_val[c] = out->alg_bytes[c]; }
  S->recs.clear();
  SCK(cudaMemsetAsync(S->read_rows, 0, 2 * sizeof(u64), S->env.stream()));
  return GCNSA_OK;
}

int gcnsa_sage_get_epoch(const gcnsa_sage* S, int64_t* epoch_out) {
  if (!S || !epoch_out) return fail(GCNSA_ERR_ARG, "NULL argument");
  *epoch_out = S->epoch;
  return GCNSA_OK;
}

int gcnsa_sage_batch_shape(const gcnsa_sage* S, int64_t* nb_out, int64_t* rows1_out) {
  if (!S || !nb_out || !rows1_out) return fail(GCNSA_ERR_ARG, "NULL argument");
  *nb_out = S->last_nb;
  *rows1_out = S->last_rows1;
  return GCNSA_OK;
}

int gcnsa_sage_batch_export(const gcnsa_sage* S, const gcnsa_sage_batch_host* dst) {
  if (!S || !dst) return fail(GCNSA_ERR_ARG, "NULL argument");
  cudaStream_t s = S->env.stream();
  const size_t nb = (size_t)S->last_nb, rows1 = (size_t)S->last_rows1;
  const size_t r1 = (size_t)S->o.fanout[0];
  if (dst->vertices && rows1) SCK(cudaMemcpyAsync(dst->vertices, S->b1, rows1 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  if (dst->count2 && nb) SCK(cudaMemcpyAsync(dst->count2, S->cnt2, nb * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  if (dst->samples1 && rows1 && r1)
    SCK(cudaMemcpyAsync(dst->samples1, S->s1, rows1 * r1 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  if (dst->count1 && rows1) SCK(cudaMemcpyAsync(dst->count1, S->cnt1, rows1 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  if (dst->hidden && rows1)
    SCK(cudaMemcpy2DAsync(dst->hidden, (size_t)S->h * sizeof(float), S->h1, (size_t)S->ldh * sizeof(float),
                          (size_t)S->h * sizeof(float), rows1, cudaMemcpyDeviceToHost, s));
  if (dst->logits && nb)
    SCK(cudaMemcpy2DAsync(dst->logits, (size_t)S->c * sizeof(float), S->logits, (size_t)S->ldc * sizeof(float),
                          (size_t)S->c * sizeof(float), nb, cudaMemcpyDeviceToHost, s));
  if (dst->dlogits && nb)
    SCK(cudaMemcpy2DAsync(dst->dlogits, (size_t)S->c * sizeof(float), S->g, (size_t)S->ldc * sizeof(float),
                          (size_t)S->c * sizeof(float), nb, cudaMemcpyDeviceToHost, s));
  if (dst->loss) SCK(cudaMemcpyAsync(dst->loss, S->loss, sizeof(float), cudaMemcpyDeviceToHost, s));
  SCK(cudaStreamSynchronize(s));
  return GCNSA_OK;
}

static int sage_param(const gcnsa_sage* S, int32_t what, int32_t layer, float** base_out, int64_t* rows, int64_t* cols,
                      int64_t* ld) {
  if (!S) return fail(GCNSA_ERR_ARG, "model is NULL");
  if (layer < 0 || layer > 1) return fail(GCNSA_ERR_ARG, "layer out of range");
  const int kind = what % 3, which = what / 3;  // kind: self, neighbour, bias; which: aggregated, working copy, gradient
  float* buf = which == 0 ? S->theta : which == 1 ? S->work : which == 2 ? S->grad : nullptr;
  if (!buf || what < 0) return fail(GCNSA_ERR_ARG, "unknown tensor id");
  const int64_t din = layer == 0 ? S->f : S->h, dout = layer == 0 ? S->h : S->c;
  const int64_t ldin = layer == 0 ? S->ldf : S->ldh, ldo = layer == 0 ? S->ldh : S->ldc;
  const int64_t w_off = layer == 0 ? S->w1_off : S->w2_off, b_off = layer == 0 ? S->b1_off : S->b2_off;
  *cols = dout; *ld = ldo;
  if (kind == 2) { *base_out = buf + b_off; *rows = 1; }
  else { *base_out = buf + w_off + (kind == 1 ? ldin * ldo : 0); *rows = din; }
  return GCNSA_OK;
}

int gcnsa_sage_get(const gcnsa_sage* S, int32_t what, int32_t layer, void* host_dst, size_t bytes) {
  float* base = nullptr;
  int64_t rows = 0, cols = 0, ld = 0;
  int rc = sage_param(S, what, layer, &base, &rows, &cols, &ld);
  if (rc) return rc;
  if (!host_dst || bytes != (size_t)(rows * cols) * sizeof(float)) return fail(GCNSA_ERR_ARG, "NULL or byte count does not match");
  SCK(cudaMemcpy2DAsync(host_dst, (size_t)cols * sizeof(float), base, (size_t)ld * sizeof(float), (size_t)cols * sizeof(float),
                        (size_t)rows, cudaMemcpyDeviceToHost, S->env.stream()));
  SCK(cudaStreamSynchronize(S->env.stream()));
  return GCNSA_OK;
}

}  // extern "C"
