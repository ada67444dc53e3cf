// C-ABI of libgcnsa: handles, device memory, and the order in which the kernels
// of one forward / backward / step are enqueued.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "internal.h"
#include "parts.h"

namespace gcnsa {

static thread_local std::string g_err;
static std::atomic<int64_t> g_launches{0};

int fail(int code, const std::string& detail) {
  g_err = detail;
  return code;
}
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
static std::atomic<int64_t> g_gemm_tc{0}, g_gemm_fallback{0};
void note_gemm_path(bool tensor_core) { (tensor_core ? g_gemm_tc : g_gemm_fallback).fetch_add(1, std::memory_order_relaxed); }

static int cuda_fail(cudaError_t e, const char* what) {
  return fail(GCNSA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define CK(call)                                          \
  do {                                                    \
    cudaError_t e_ = (call);                              \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);   \
  } while (0)
#define CKL(call)                                                       \
  do {                                                                  \
    int e_ = (call);                                                    \
    if (e_ != 0) return cuda_fail((cudaError_t)e_, #call);              \
  } while (0)

static int check_device(const gcnsa_env* env) {
  if (!env) return fail(GCNSA_ERR_ARG, "env is NULL");
  if ((env->alloc == nullptr) != (env->free == nullptr)) return fail(GCNSA_ERR_ARG, "alloc and free must come together");
  int count = 0;
  cudaError_t e = cudaGetDeviceCount(&count);
  if (e != cudaSuccess || count == 0) {
    cudaGetLastError();
    return fail(GCNSA_ERR_CUDA, "no CUDA device: this library has no CPU fallback");
  }
  if (env->device < 0 || env->device >= count) return fail(GCNSA_ERR_ARG, "device index out of range");
  CK(cudaSetDevice(env->device));
  cudaDeviceProp prop;
  CK(cudaGetDeviceProperties(&prop, env->device));
  if (prop.major != 10) return fail(GCNSA_ERR_UNSUPPORTED_ARCH, "kernels are built for sm_100a only");
  return GCNSA_OK;
}

}  // namespace gcnsa

using namespace gcnsa;

extern "C" int64_t gcnsa_launch_count(void);

struct gcnsa_model {
  Env env;
  gcnsa_model_opts o{};
  int32_t L = 0, m = 0;
  int64_t n_max = 0, count = 0;  // count = floats in the flat parameter buffer
  int64_t w_off[GCNSA_MAX_LAYERS], b_off[GCNSA_MAX_LAYERS], w_ld[GCNSA_MAX_LAYERS];
  bool transform_first[GCNSA_MAX_LAYERS];
  float *theta = nullptr, *gsum = nullptr, *am = nullptr, *av = nullptr;
  // parameter-averaging mode: Adam moments per partition ([m x count]) and the running mean of the partitions' parameters
  float *am_parts = nullptr, *av_parts = nullptr, *theta_acc = nullptr;
  int32_t state_p = 0;
  bool all_rows_once = false;  // set by gcnsa_evaluate: the next forward computes every logit row
  double* adam_state = nullptr;  // device: step count t and the two bias corrections of Adam
  // recorded epoch (epoch_graph): valid for one partitions object and one loss pointer
  cudaGraphExec_t graph_exec = nullptr;
  uint64_t graph_parts_uid = 0;
  const void* graph_loss = nullptr;
  int graph_kernels = 0;  // kernel launches one replay stands for
  bool graph_off = false;
  // cache_ax: A_hat X of every partition of one partitions object, kept while the feature rows stay the same
  std::vector<float*> ax;
  std::vector<int64_t> ax_version;  // x_version of the partition the product was computed from (0 = none yet)
  uint64_t ax_uid = 0;
  const float* s0_used = nullptr;   // A_hat H^0 the latest forward used (the cached one or S[0])
  float* H[GCNSA_MAX_LAYERS + 1] = {nullptr};  // H[l], l >= 1
  float* S[GCNSA_MAX_LAYERS] = {nullptr};      // A_hat H^{l-1} of layers that aggregate first
  float *tmp_a = nullptr, *tmp_b = nullptr, *dlogits = nullptr, *loss_parts = nullptr;
  // evaluation buffers (allocated on first gcnsa_evaluate)
  int32_t *ev_pred = nullptr, *ev_hits = nullptr;
  uint8_t* ev_mask = nullptr;
  void *ws = nullptr, *sc = nullptr;
  size_t ws_bytes = 0, sc_bytes = 0;
  int64_t ld_max = 0;
  int32_t last_forward = -1, accumulated = 0;
  int64_t last_n = 0;
  int64_t t = 0;
  std::vector<void*> owned;
  void* dalloc(size_t bytes) {
    void* p = env.alloc(bytes);
    if (p) owned.push_back(p);
    return p;
  }
  // optional per-kernel timing
  struct Rec { int cat; double bytes, flops, l1, bytes_val; int64_t launches; };
  bool prof_on = false;
  std::vector<cudaEvent_t> ev;  // pairs, reused
  std::vector<Rec> recs;
  int64_t launches_mark = 0;
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
  void prof_end(int cat, double bytes, double flops, double l1 = -1.0, double bytes_val = -1.0) {
    if (!prof_on) return;
    cudaEventRecord(ev[recs.size() * 2 + 1], env.stream());
    recs.push_back({cat, bytes, flops, l1 < 0.0 ? bytes : l1, bytes_val < 0.0 ? bytes : bytes_val,
                    gcnsa_launch_count() - launches_mark});
  }
};

// Memory accounting of one sparse product over `rows` result rows, `nnz` stored entries and `n_src` source rows
// that are referenced, at width f.  bytes: what must cross HBM once (row pointers, column indices, values - none
// when the normalization is factored out: then one scale per row -, one read of the source rows, one write of the
// result, one read of a ReLU mask).  l1: what the SMs pull through the L1 data path: the same, except that every
// stored entry gathers its own source row (4 f nnz instead of 4 f n_src).
// bytes_val: `bytes` with 8 bytes per stored entry (index + value) whether or not the kernel reads values.
struct SpmmCost { double bytes, l1, flops, bytes_val; };
static SpmmCost spmm_cost(int64_t rows, int64_t n_src, int64_t nnz, int64_t f, bool values, bool mask = false) {
  const double idx = 4.0 * (double)(rows + 1) + (values ? 8.0 * (double)nnz : 4.0 * (double)nnz + 4.0 * (double)rows);
  const double out = 4.0 * (double)f * (double)rows * (mask ? 2.0 : 1.0);
  SpmmCost c;
  c.bytes = idx + 4.0 * (double)f * (double)n_src + out;
  c.l1 = idx + 4.0 * (double)f * (double)nnz + out;
  c.flops = 2.0 * (double)nnz * (double)f;
  c.bytes_val = 4.0 * (double)(rows + 1) + 8.0 * (double)nnz + 4.0 * (double)f * (double)n_src + out;
  return c;
}
static double gemm_bytes(int64_t m, int64_t n, int64_t k) { return 4.0 * ((double)m * k + (double)k * n + (double)m * n); }
#define PROF(M, cat, bytes, flops, call) \
  do {                                   \
    (M)->prof_begin();                   \
    CKL(call);                           \
    (M)->prof_end(cat, bytes, flops);    \
  } while (0)
#define PROF_SPMM(M, cost, call)                             \
  do {                                                       \
    const SpmmCost c_ = (cost);                              \
    (M)->prof_begin();                                       \
    CKL(call);                                               \
    (M)->prof_end(0, c_.bytes, c_.flops, c_.l1, c_.bytes_val); \
  } while (0)

extern "C" {

const char* gcnsa_strerror(int code) {
  switch (code) {
    case GCNSA_OK: return "ok";
    case GCNSA_ERR_ARG: return "invalid argument";
    case GCNSA_ERR_NOT_SYMMETRIC: return "graph is not symmetric";
    case GCNSA_ERR_SELF_LOOP_OR_DUP: return "graph has a self-loop or a repeated edge";
    case GCNSA_ERR_LABEL_RANGE: return "label or partition id out of range";
    case GCNSA_ERR_OOM: return "out of memory";
    case GCNSA_ERR_ORDER: return "calls in the wrong order";
    case GCNSA_ERR_CUDA: return "CUDA error";
    case GCNSA_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    case GCNSA_ERR_TOO_LARGE: return "partition exceeds int32 indexing";
    default: return "unknown error";
  }
}
const char* gcnsa_last_error(void) { return g_err.c_str(); }
int64_t gcnsa_launch_count(void) { return g_launches.load(); }
int gcnsa_gemm_path_counts(int64_t* tensor_core, int64_t* fp32_fallback) {
  if (!tensor_core || !fp32_fallback) return fail(GCNSA_ERR_ARG, "NULL argument");
  *tensor_core = g_gemm_tc.load();
  *fp32_fallback = g_gemm_fallback.load();
  return GCNSA_OK;
}
void gcnsa_model_opts_default(gcnsa_model_opts* o) {
  if (!o) return;
  std::memset(o, 0, sizeof(*o));
  o->n_layers = 2;
  o->use_bias = 1;
  o->lr = 0.02f; o->beta1 = 0.9f; o->beta2 = 0.999f; o->eps = 1e-8f;
  o->gemm_mode = GCNSA_GEMM_TF32X3;
  o->agg_mode = GCNSA_AGG_GRAD_AVG;
  o->loss_rows_only = 1;
  o->epoch_graph = 1;
  o->factored_norm = 1;
  o->cache_ax = 0;
}

// ------------------------------------------------------------------ parts ---
int gcnsa_parts_destroy(gcnsa_parts* parts) {
  if (!parts) return GCNSA_OK;
  cudaStreamSynchronize(parts->env.stream());
  if (parts->copy_stream) {
    cudaStreamSynchronize(parts->copy_stream);
    cudaStreamDestroy(parts->copy_stream);
  }
  for (cudaEvent_t e : parts->ready) cudaEventDestroy(e);
  for (cudaEvent_t e : parts->consumed) cudaEventDestroy(e);
  for (void* p : parts->owned) parts->env.release(p);
  delete parts;
  return GCNSA_OK;
}

static int upload(gcnsa_parts* P, void** dst, const void* src, size_t bytes) {
  *dst = P->dalloc(bytes);
  if (!*dst) return fail(GCNSA_ERR_OOM, "device allocation failed");
  if (bytes) CK(cudaMemcpyAsync(*dst, src, bytes, cudaMemcpyHostToDevice, P->env.stream()));
  return GCNSA_OK;
}

static int build_failed(gcnsa_parts* P, int rc) {
  std::string keep = g_err;
  gcnsa_parts_destroy(P);
  g_err = keep;
  return rc;
}

int gcnsa_build_partitions(const gcnsa_env* env, const gcnsa_graph* g, const gcnsa_part_opts* opts, gcnsa_parts** out) {
  if (!out) return fail(GCNSA_ERR_ARG, "out is NULL");
  *out = nullptr;
  int rc = check_build_args(g, opts);
  if (rc) return rc;
  HostBuild hb;
  const bool on_host = opts->builder == GCNSA_BUILD_HOST;
  if (on_host) {
    rc = build_host(g, opts, &hb);
    if (rc) return rc;
  }
  rc = check_device(env);
  if (rc) {
    // without a usable device an invalid graph is still reported as such (checked on the host cores)
    if (!on_host) {
      const std::string keep = g_err;
      const int v = validate_graph_host(g);
      if (v) return v;
      g_err = keep;
    }
    return rc;
  }
  gcnsa_parts* P = new (std::nothrow) gcnsa_parts();
  if (!P) return fail(GCNSA_ERR_OOM, "host allocation failed");
  P->env.e = *env;
  P->m = opts->m; P->f = g->f; P->c = g->c; P->n = g->n; P->ldx = GCNSA_LD(g->f);
  P->builder = opts->builder;
  P->x_version.assign((size_t)opts->m, 1);
  static std::atomic<uint64_t> next_uid{1};
  P->uid = next_uid.fetch_add(1);
  if (!on_host) {
    rc = build_device(P, g, opts);
    if (rc) return build_failed(P, rc);
    *out = P;
    return GCNSA_OK;
  }
  P->part.swap(hb.part);
  P->parts.resize((size_t)opts->m);
  cudaStream_t s = P->env.stream();
  std::vector<float> xs;
  std::vector<int32_t> ys, deg;
  std::vector<uint8_t> ms;
  for (int32_t p = 0; p < opts->m && rc == GCNSA_OK; ++p) {
    HostPart& hp = hb.parts[p];
    DevPart& d = P->parts[p];
    d.info.n_owned = hp.n_owned; d.info.n_halo = hp.n_halo; d.info.n = hp.n; d.info.nnz = hp.nnz;
    d.info.nts = hp.nts; d.info.n_train = hp.n_train; d.info.max_depth = hp.max_depth;
    d.n_long = hp.n_long; d.t_n_long = hp.t_n_long;
    d.tm_n_long = hp.tm_n_long; d.tm_nnz = (int64_t)hp.tm_col.size();
    d.m_n_long = hp.m_n_long; d.m_nnz = hp.m_nnz;
    d.members.swap(hp.members);
    d.depth.swap(hp.depth);
    P->n_max = std::max(P->n_max, hp.n);
    const size_t n = (size_t)hp.n, nnz = (size_t)hp.nnz;
    // features, labels and mask in partition order (pad columns zero)
    xs.assign(n * (size_t)P->ldx, 0.f);
    ys.resize(n); ms.resize(n); deg.resize(n);
    {
      const int64_t chunk = 2048, n_chunks = ((int64_t)n + chunk - 1) / chunk;
      std::atomic<int64_t> next{0};
      auto work = [&] {
        for (;;) {
          const int64_t ci = next.fetch_add(1);
          if (ci >= n_chunks) break;
          for (int64_t i = ci * chunk; i < std::min<int64_t>((int64_t)n, (ci + 1) * chunk); ++i)
            std::memcpy(&xs[(size_t)i * P->ldx], g->x + d.members[i] * g->ldx, sizeof(float) * (size_t)g->f);
        }
      };
      int nt = (int)std::min<int64_t>(std::max(1u, std::thread::hardware_concurrency()), 16);
      std::vector<std::thread> th;
      for (int t = 1; t < nt; ++t) th.emplace_back(work);
      work();
      for (auto& t : th) t.join();
    }
    for (size_t i = 0; i < n; ++i) {
      ys[i] = g->y[d.members[i]];
      const bool carries = opts->loss_on_halo || (int64_t)i < hp.n_owned;
      ms[i] = (carries && g->train_mask[d.members[i]]) ? 1 : 0;
      deg[i] = hp.rowptr[i + 1] - hp.rowptr[i];
    }
    void* ddeg = nullptr;
#define UP(field, vec, type) if (rc == GCNSA_OK) rc = upload(P, (void**)&d.field, vec.data(), vec.size() * sizeof(type))
    UP(rowptr, hp.rowptr, int32_t); UP(col, hp.col, int32_t); UP(t_rowptr, hp.t_rowptr, int32_t);
    UP(t_col, hp.t_col, int32_t); UP(order, hp.order, int32_t); UP(t_order, hp.t_order, int32_t);
    UP(x, xs, float); UP(y, ys, int32_t); UP(mask, ms, uint8_t);
    UP(m_order, hp.m_order, int32_t);
    UP(tm_rowptr, hp.tm_rowptr, int32_t); UP(tm_col, hp.tm_col, int32_t); UP(tm_order, hp.tm_order, int32_t);
#undef UP
    if (rc == GCNSA_OK) rc = upload(P, &ddeg, deg.data(), n * sizeof(int32_t));
    if (rc == GCNSA_OK) {
      d.val = (float*)P->dalloc(std::max<size_t>(nnz, 1) * sizeof(float));
      d.t_val = (float*)P->dalloc(std::max<size_t>(nnz, 1) * sizeof(float));
      d.tm_val = (float*)P->dalloc(std::max<size_t>((size_t)d.tm_nnz, 1) * sizeof(float));
      d.dinv = (float*)P->dalloc(std::max<size_t>(n, 1) * sizeof(float));
      if (!d.val || !d.t_val || !d.tm_val || !d.dinv) rc = fail(GCNSA_ERR_OOM, "device allocation failed");
    }
    if (rc == GCNSA_OK) {
      // entry (i, j) of A_hat and entry (j, i) of its transpose are both
      // 1 / sqrt(d_i d_j) with d the row lengths of A + I: one degree array serves both
      int e1 = launch_normalize(s, hp.n, d.rowptr, d.col, (const int32_t*)ddeg, d.val);
      int e2 = launch_normalize(s, hp.n, d.t_rowptr, d.t_col, (const int32_t*)ddeg, d.t_val);
      if (!e2) e2 = launch_normalize(s, hp.n, d.tm_rowptr, d.tm_col, (const int32_t*)ddeg, d.tm_val);
      if (!e2) e2 = launch_inv_sqrt_degree(s, hp.n, (const int32_t*)ddeg, d.dinv);
      if (e1 || e2) rc = cuda_fail((cudaError_t)(e1 ? e1 : e2), "normalize");
    }
    // host staging vectors are reused: wait for the copies of this partition
    if (rc == GCNSA_OK) {
      cudaError_t e = cudaStreamSynchronize(s);
      if (e != cudaSuccess) rc = cuda_fail(e, "cudaStreamSynchronize");
    }
  }
  if (rc != GCNSA_OK) return build_failed(P, rc);
  *out = P;
  return GCNSA_OK;
}

int gcnsa_parts_count(const gcnsa_parts* parts) { return parts ? parts->m : GCNSA_ERR_ARG; }

int gcnsa_parts_info(const gcnsa_parts* parts, int32_t p, gcnsa_part_info* out) {
  if (!parts || !out || p < 0 || p >= parts->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  *out = parts->parts[p].info;
  return GCNSA_OK;
}

int gcnsa_parts_assignment(const gcnsa_parts* parts, int32_t* part_host) {
  if (!parts || !part_host) return fail(GCNSA_ERR_ARG, "NULL argument");
  std::memcpy(part_host, parts->part.data(), parts->part.size() * sizeof(int32_t));
  return GCNSA_OK;
}

int gcnsa_parts_export(const gcnsa_parts* parts, int32_t p, const gcnsa_part_host* dst) {
  if (!parts || !dst || p < 0 || p >= parts->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const DevPart& d = parts->parts[p];
  cudaStream_t s = parts->env.stream();
  const size_t n = (size_t)d.info.n, nnz = (size_t)d.info.nnz;
#define DOWN(field, count, type) \
  if (dst->field) CK(cudaMemcpyAsync(dst->field, d.field, (count) * sizeof(type), cudaMemcpyDeviceToHost, s))
  DOWN(rowptr, n + 1, int32_t); DOWN(col, nnz, int32_t); DOWN(val, nnz, float);
  DOWN(t_rowptr, n + 1, int32_t); DOWN(t_col, nnz, int32_t); DOWN(t_val, nnz, float);
#undef DOWN
  if (dst->members) std::memcpy(dst->members, d.members.data(), n * sizeof(int64_t));
  if (dst->depth) std::memcpy(dst->depth, d.depth.data(), d.depth.size() * sizeof(int32_t));
  CK(cudaStreamSynchronize(s));
  return GCNSA_OK;
}

int gcnsa_parts_export_schedule(const gcnsa_parts* parts, int32_t p, gcnsa_part_schedule_info* info,
                                const gcnsa_part_schedule_host* dst) {
  if (!parts || p < 0 || p >= parts->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const DevPart& d = parts->parts[p];
  if (info) {
    info->n_long = d.n_long; info->t_n_long = d.t_n_long; info->m_n_long = d.m_n_long; info->tm_n_long = d.tm_n_long;
    info->m_nnz = d.m_nnz; info->tm_nnz = d.tm_nnz;
  }
  if (!dst) return GCNSA_OK;
  cudaStream_t s = parts->env.stream();
  const size_t n = (size_t)d.info.n;
#define DOWN(field, count, type) \
  if (dst->field && (count)) CK(cudaMemcpyAsync(dst->field, d.field, (count) * sizeof(type), cudaMemcpyDeviceToHost, s))
  DOWN(order, n, int32_t); DOWN(t_order, n, int32_t); DOWN(m_order, (size_t)d.info.n_train, int32_t);
  DOWN(tm_rowptr, n + 1, int32_t); DOWN(tm_col, (size_t)d.tm_nnz, int32_t); DOWN(tm_order, n, int32_t);
  DOWN(mask, n, uint8_t); DOWN(y, n, int32_t);
#undef DOWN
  CK(cudaStreamSynchronize(s));
  return GCNSA_OK;
}

int gcnsa_parts_get_features(const gcnsa_parts* parts, int32_t p, float* x_host) {
  if (!parts || !x_host || p < 0 || p >= parts->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const DevPart& d = parts->parts[p];
  if (d.info.n == 0) return GCNSA_OK;
  CK(cudaMemcpy2DAsync(x_host, (size_t)parts->f * sizeof(float), d.x, (size_t)parts->ldx * sizeof(float),
                       (size_t)parts->f * sizeof(float), (size_t)d.info.n, cudaMemcpyDeviceToHost, parts->env.stream()));
  CK(cudaStreamSynchronize(parts->env.stream()));
  return GCNSA_OK;
}

int gcnsa_parts_set_features(gcnsa_parts* parts, int32_t p, const float* x_host) {
  if (!parts || !x_host || p < 0 || p >= parts->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  DevPart& d = parts->parts[p];
  CK(cudaMemcpy2DAsync(d.x, (size_t)parts->ldx * sizeof(float), x_host, (size_t)parts->f * sizeof(float),
                       (size_t)parts->f * sizeof(float), (size_t)d.info.n, cudaMemcpyHostToDevice, parts->env.stream()));
  parts->x_version[p] += 1;
  return GCNSA_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ model ---
extern "C" {

int gcnsa_model_destroy(gcnsa_model* model) {
  if (!model) return GCNSA_OK;
  cudaStreamSynchronize(model->env.stream());
  for (void* p : model->owned) model->env.release(p);
  for (cudaEvent_t e : model->ev) cudaEventDestroy(e);
  if (model->graph_exec) cudaGraphExecDestroy(model->graph_exec);
  delete model;
  return GCNSA_OK;
}

static int copy_param(const gcnsa_model* M, float* base, int32_t layer, bool is_w, void* host, size_t bytes, bool to_host) {
  const int64_t rows = is_w ? M->o.dims[layer] : 1, cols = M->o.dims[layer + 1];
  if (bytes != (size_t)(rows * cols) * sizeof(float)) return fail(GCNSA_ERR_ARG, "byte count does not match the tensor");
  float* d = base + (is_w ? M->w_off[layer] : M->b_off[layer]);
  const size_t dpitch = (size_t)(is_w ? M->w_ld[layer] : cols) * sizeof(float), hpitch = (size_t)cols * sizeof(float);
  if (to_host) CK(cudaMemcpy2DAsync(host, hpitch, d, dpitch, hpitch, (size_t)rows, cudaMemcpyDeviceToHost, M->env.stream()));
  else CK(cudaMemcpy2DAsync(d, dpitch, host, hpitch, hpitch, (size_t)rows, cudaMemcpyHostToDevice, M->env.stream()));
  CK(cudaStreamSynchronize(M->env.stream()));
  return GCNSA_OK;
}

int gcnsa_model_create(const gcnsa_env* env, const gcnsa_parts* parts, const gcnsa_model_opts* opts,
                       const float* const* w0, const float* const* b0, gcnsa_model** out) {
  if (!out) return fail(GCNSA_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (!env || !parts || !opts || !w0) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (opts->n_layers < 1 || opts->n_layers > GCNSA_MAX_LAYERS) return fail(GCNSA_ERR_ARG, "n_layers out of range");
  for (int l = 0; l <= opts->n_layers; ++l)
    if (opts->dims[l] < 1) return fail(GCNSA_ERR_ARG, "layer width < 1");
  if (opts->dims[0] != parts->f || opts->dims[opts->n_layers] != parts->c)
    return fail(GCNSA_ERR_ARG, "dims[0] must equal f and dims[L] must equal c of the partitions");
  if (opts->gemm_mode != GCNSA_GEMM_FP32 && opts->gemm_mode != GCNSA_GEMM_TF32X3 && opts->gemm_mode != GCNSA_GEMM_TF32)
    return fail(GCNSA_ERR_ARG, "unknown gemm_mode");
  if (opts->agg_mode != GCNSA_AGG_GRAD_AVG && opts->agg_mode != GCNSA_AGG_PARAM_AVG)
    return fail(GCNSA_ERR_ARG, "unknown agg_mode");
  if (!(opts->lr > 0.f) || !(opts->beta1 >= 0.f && opts->beta1 < 1.f) || !(opts->beta2 >= 0.f && opts->beta2 < 1.f) ||
      !(opts->eps > 0.f))
    return fail(GCNSA_ERR_ARG, "Adam hyper-parameters out of range");
  int rc = check_device(env);
  if (rc) return rc;
  gcnsa_model* M = new (std::nothrow) gcnsa_model();
  if (!M) return fail(GCNSA_ERR_OOM, "host allocation failed");
  M->env.e = *env;
  M->o = *opts;
  M->L = opts->n_layers;
  M->m = parts->m;
  M->n_max = std::max<int64_t>(parts->n_max, 1);
  int64_t off = 0;
  M->ld_max = 0;
  for (int l = 0; l < M->L; ++l) {
    const int64_t din = opts->dims[l], dout = opts->dims[l + 1];
    M->w_ld[l] = GCNSA_LD(dout);
    M->w_off[l] = off; off += (din * M->w_ld[l] + 63) / 64 * 64;
    M->b_off[l] = off; off += (M->w_ld[l] + 63) / 64 * 64;
    M->transform_first[l] = dout <= din;  // multiply by W first when the layer does not widen
    if (l == 0 && opts->cache_ax) M->transform_first[l] = false;  // (A_hat X) W with A_hat X kept across epochs
    M->ld_max = std::max<int64_t>(M->ld_max, std::max<int64_t>(GCNSA_LD(din), GCNSA_LD(dout)));
  }
  M->count = off;
  auto fail_free = [&](int code) {
    std::string keep = g_err;
    gcnsa_model_destroy(M);
    g_err = keep;
    return code;
  };
  const size_t pbytes = (size_t)off * sizeof(float);
  M->theta = (float*)M->dalloc(pbytes); M->gsum = (float*)M->dalloc(pbytes);
  M->am = (float*)M->dalloc(pbytes);    M->av = (float*)M->dalloc(pbytes);
  const size_t act = (size_t)M->n_max * (size_t)M->ld_max * sizeof(float);
  M->tmp_a = (float*)M->dalloc(act); M->tmp_b = (float*)M->dalloc(act);
  M->dlogits = (float*)M->dalloc((size_t)M->n_max * GCNSA_LD(parts->c) * sizeof(float));
  M->loss_parts = (float*)M->dalloc((size_t)(M->m + 1) * sizeof(float));
  M->adam_state = (double*)M->dalloc(4 * sizeof(double));
  bool ok = M->theta && M->gsum && M->am && M->av && M->tmp_a && M->tmp_b && M->dlogits && M->loss_parts && M->adam_state;
  size_t ws = 0, sc = softmax_ce_scratch(M->n_max);
  for (int l = 0; l < M->L && ok; ++l) {
    const int64_t din = opts->dims[l], dout = opts->dims[l + 1];
    M->H[l + 1] = (float*)M->dalloc((size_t)M->n_max * GCNSA_LD(dout) * sizeof(float));
    ok = ok && M->H[l + 1];
    if (!M->transform_first[l]) {
      M->S[l] = (float*)M->dalloc((size_t)M->n_max * GCNSA_LD(din) * sizeof(float));
      ok = ok && M->S[l];
    }
    ws = std::max(ws, gemm_workspace(opts->gemm_mode, 1, 0, din, dout, M->n_max));
    ws = std::max(ws, gemm_workspace(opts->gemm_mode, 0, 0, M->n_max, dout, din));
    ws = std::max(ws, gemm_workspace(opts->gemm_mode, 0, 1, M->n_max, din, dout));
    sc = std::max(sc, colsum_scratch(M->n_max, (int32_t)dout));
    sc = std::max(sc, gemm_colsum_scratch(M->n_max, (int32_t)din));  // the fused bias gradient of the layer below
  }
  if (ok && opts->cache_ax) {
    M->ax.assign((size_t)parts->m, nullptr);
    M->ax_version.assign((size_t)parts->m, 0);
    M->ax_uid = parts->uid;
    for (int32_t p = 0; p < parts->m && ok; ++p) {
      const size_t bytes = (size_t)std::max<int64_t>(parts->parts[p].info.n, 1) * (size_t)parts->ldx * sizeof(float);
      M->ax[p] = (float*)M->dalloc(bytes);
      ok = M->ax[p] != nullptr;
      if (ok) cudaMemsetAsync(M->ax[p], 0, bytes, M->env.stream());
    }
  }
  if (ok && opts->agg_mode == GCNSA_AGG_PARAM_AVG) {
    const size_t pb = (size_t)M->count * sizeof(float);
    M->am_parts = (float*)M->dalloc(pb * M->m);
    M->av_parts = (float*)M->dalloc(pb * M->m);
    M->theta_acc = (float*)M->dalloc(pb);
    ok = M->am_parts && M->av_parts && M->theta_acc;
    if (ok) {
      cudaMemsetAsync(M->am_parts, 0, pb * M->m, M->env.stream());
      cudaMemsetAsync(M->av_parts, 0, pb * M->m, M->env.stream());
      cudaMemsetAsync(M->theta_acc, 0, pb, M->env.stream());
    }
  }
  if (ok) {
    M->ws_bytes = ws; M->sc_bytes = sc;
    M->ws = M->dalloc(std::max<size_t>(ws, 256)); M->sc = M->dalloc(std::max<size_t>(sc, 256));
    ok = M->ws && M->sc;
  }
  if (!ok) return fail_free(fail(GCNSA_ERR_OOM, "device allocation failed"));
  cudaStream_t s = M->env.stream();
  cudaError_t e = cudaMemsetAsync(M->theta, 0, pbytes, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->gsum, 0, pbytes, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->am, 0, pbytes, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->av, 0, pbytes, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->tmp_a, 0, act, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->tmp_b, 0, act, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->dlogits, 0, (size_t)M->n_max * GCNSA_LD(parts->c) * sizeof(float), s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->loss_parts, 0, (size_t)(M->m + 1) * sizeof(float), s);
  if (e == cudaSuccess) e = cudaMemsetAsync(M->adam_state, 0, 4 * sizeof(double), s);
  for (int l = 0; l < M->L && e == cudaSuccess; ++l) {
    e = cudaMemsetAsync(M->H[l + 1], 0, (size_t)M->n_max * GCNSA_LD(opts->dims[l + 1]) * sizeof(float), s);
    if (e == cudaSuccess && M->S[l])
      e = cudaMemsetAsync(M->S[l], 0, (size_t)M->n_max * GCNSA_LD(opts->dims[l]) * sizeof(float), s);
  }
  if (e != cudaSuccess) return fail_free(cuda_fail(e, "cudaMemsetAsync"));
  for (int l = 0; l < M->L; ++l) {
    if (!w0[l]) return fail_free(fail(GCNSA_ERR_ARG, "w0[l] is NULL"));
    rc = copy_param(M, M->theta, l, true, (void*)w0[l], (size_t)opts->dims[l] * opts->dims[l + 1] * sizeof(float), false);
    if (rc == GCNSA_OK && b0 && b0[l])
      rc = copy_param(M, M->theta, l, false, (void*)b0[l], (size_t)opts->dims[l + 1] * sizeof(float), false);
    if (rc) return fail_free(rc);
  }
  *out = M;
  return GCNSA_OK;
}

// cache_ax: (re)computes A_hat X of partition p if its feature rows changed since the cached product was made
static int ensure_ax(gcnsa_model* M, const gcnsa_parts* P, int32_t p) {
  if (M->ax_version[p] == P->x_version[p]) return GCNSA_OK;
  const DevPart& d = P->parts[p];
  const int32_t din = M->o.dims[0];
  PROF_SPMM(M, spmm_cost(d.info.n, d.info.n, d.info.nnz, din, true),
       launch_spmm(M->env.e.stream, d.info.n, d.rowptr, d.col, d.val, nullptr, d.order, d.n_long, d.x, P->ldx, din,
                   GCNSA_EPI_NONE, nullptr, 0, M->ax[p], P->ldx, SpmmBounds{d.info.n, d.info.n, d.info.nnz}));
  M->ax_version[p] = P->x_version[p];
  return GCNSA_OK;
}

int gcnsa_forward(gcnsa_model* M, const gcnsa_parts* P, int32_t p, float* loss_dev) {
  if (!M || !P || p < 0 || p >= P->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  if (P->m != M->m || P->f != M->o.dims[0] || P->c != M->o.dims[M->L] || P->n_max > M->n_max)
    return fail(GCNSA_ERR_ARG, "model was created for other partitions");
  const DevPart& d = P->parts[p];
  void* s = M->env.e.stream;
  const int64_t n = d.info.n, nnz = d.info.nnz;
  const float* h = d.x;
  int64_t ldh = P->ldx;
  const bool fact = M->o.factored_norm != 0;
  const float* rs = fact ? d.dinv : nullptr;
  for (int l = 0; l < M->L; ++l) {
    const int32_t din = M->o.dims[l], dout = M->o.dims[l + 1];
    const bool last = l == M->L - 1;
    const float* bias = M->o.use_bias ? M->theta + M->b_off[l] : nullptr;
    const int epi = last ? (bias ? GCNSA_EPI_BIAS : GCNSA_EPI_NONE) : GCNSA_EPI_BIAS_RELU;
    const float* w = M->theta + M->w_off[l];
    const int64_t ldo = GCNSA_LD(dout);
    if (M->transform_first[l]) {
      // factored_norm: A_hat T = diag(dinv) (A + I) (diag(dinv) T): the GEMM's epilogue scales the rows of T and
      // the product reads no values
      PROF(M, 1, gemm_bytes(n, dout, din), 2.0 * n * dout * din,
           launch_gemm(s, M->o.gemm_mode, 0, 0, n, dout, din, h, ldh, w, M->w_ld[l], M->tmp_a, ldo, 0,
                       fact ? GCNSA_EPI_ROWSCALE : GCNSA_EPI_NONE, fact ? d.dinv : nullptr, 0, M->ws, M->ws_bytes));
      const float* val = fact ? nullptr : d.val;
      if (last && M->o.loss_rows_only && !M->all_rows_once) {
        // training reads the logits of the rows that carry loss only: the other rows are not computed
        PROF_SPMM(M, spmm_cost(d.info.n_train, n, d.m_nnz, dout, !fact),
             launch_spmm(s, d.info.n_train, d.rowptr, d.col, val, rs, d.m_order, d.m_n_long, M->tmp_a, ldo, dout, epi, bias, 0,
                         M->H[l + 1], ldo, SpmmBounds{n, n, nnz}));
      } else {
        PROF_SPMM(M, spmm_cost(n, n, nnz, dout, !fact),
             launch_spmm(s, n, d.rowptr, d.col, val, rs, d.order, d.n_long, M->tmp_a, ldo, dout, epi, bias, 0, M->H[l + 1], ldo, SpmmBounds{n, n, nnz}));
      }
    } else {
      const float* agg = M->S[l];
      if (l == 0 && M->o.cache_ax && P->uid == M->ax_uid) {
        // A_hat X does not change between epochs: computed when the feature rows were (re)written, reused otherwise
        int rc = ensure_ax(M, P, p);
        if (rc) return rc;
        agg = M->ax[p];
      } else {
        PROF_SPMM(M, spmm_cost(n, n, nnz, din, true),
             launch_spmm(s, n, d.rowptr, d.col, d.val, nullptr, d.order, d.n_long, h, ldh, din, GCNSA_EPI_NONE, nullptr, 0, M->S[l], ldh, SpmmBounds{n, n, nnz}));
      }
      if (l == 0) M->s0_used = agg;
      PROF(M, 1, gemm_bytes(n, dout, din), 2.0 * n * dout * din,
           launch_gemm(s, M->o.gemm_mode, 0, 0, n, dout, din, agg, ldh, w, M->w_ld[l], M->H[l + 1], ldo, 0, epi, bias,
                       0, M->ws, M->ws_bytes));
    }
    h = M->H[l + 1];
    ldh = ldo;
  }
  const int64_t ldc = GCNSA_LD(P->c);
  PROF(M, 2, 8.0 * n * P->c + 5.0 * n, 0.0,
       launch_softmax_ce(s, n, P->c, h, ldc, d.y, d.mask, d.info.n_train, M->loss_parts + p, M->dlogits, ldc, M->sc));
  if (loss_dev)
    CK(cudaMemcpyAsync(loss_dev, M->loss_parts + p, sizeof(float), cudaMemcpyDeviceToDevice, (cudaStream_t)s));
  M->last_forward = p;
  M->last_n = n;
  return GCNSA_OK;
}

int gcnsa_backward(gcnsa_model* M, const gcnsa_parts* P, int32_t p) {
  if (!M || !P || p < 0 || p >= P->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  if (M->last_forward != p) return fail(GCNSA_ERR_ORDER, "gcnsa_backward needs gcnsa_forward on the same partition first");
  if (M->accumulated >= M->m) return fail(GCNSA_ERR_ORDER, "all M partitions are accumulated already: call gcnsa_step");
  const DevPart& d = P->parts[p];
  void* s = M->env.e.stream;
  const int64_t n = d.info.n, nnz = d.info.nnz;
  const float* g = M->dlogits;  // gradient w.r.t. Z^l, [n x LD(dims[l+1])]
  const bool fact = M->o.factored_norm != 0;
  const float* rs = fact ? d.dinv : nullptr;
  bool bias_done = false, g_scaled = false;  // what the producer of g has done for this layer already
  for (int l = M->L - 1; l >= 0; --l) {
    const int32_t din = M->o.dims[l], dout = M->o.dims[l + 1];
    const int64_t ldo = GCNSA_LD(dout), ldi = GCNSA_LD(din);
    const float* hprev = l == 0 ? d.x : M->H[l];
    const float* w = M->theta + M->w_off[l];
    float* gw = M->gsum + M->w_off[l];
    // with factored_norm the products of the layers that multiply by W first read diag(dinv) G: the column-sum
    // kernel, which reads every element of G anyway, writes that copy to tmp_a (G itself below the last layer)
    bool scaled = false;
    if (bias_done) {  // the masked product of the layer above has added the column sums (and scaled g) already
      scaled = g_scaled;
    } else if (M->o.use_bias) {
      if (fact && M->transform_first[l]) {
        PROF(M, 2, 12.0 * n * dout, 0.0,
             launch_colsum_scaled(s, n, dout, g, ldo, M->gsum + M->b_off[l], 1, M->sc, d.dinv, M->tmp_a, ldo));
        scaled = true;
      } else {
        PROF(M, 2, 4.0 * n * dout, 0.0, launch_colsum(s, n, dout, g, ldo, M->gsum + M->b_off[l], 1, M->sc));
      }
    }
    if (M->transform_first[l]) {
      // Q = A_hat^T G;  dW += H^{l-1}^T Q;  G^{l-1} = (Q W^T) .* [H^{l-1} > 0]
      if (fact) {
        // A_hat^T G = diag(dinv) (A + I)^T (diag(dinv) G): the scaled copy is in tmp_a (free at this point; for
        // the layers below the last, G is tmp_a itself and was scaled in place after its column sums were taken)
        if (!scaled) PROF(M, 2, 8.0 * n * dout, 0.0, launch_scale_rows(s, n, dout, d.dinv, g, ldo, M->tmp_a, ldo));
        g = M->tmp_a;
      }
      if (l == M->L - 1) {
        // the logit gradient has zero rows outside T_p: only the non-zeros whose column carries loss contribute
        PROF_SPMM(M, spmm_cost(n, d.info.n_train, d.tm_nnz, dout, !fact),
             launch_spmm(s, n, d.tm_rowptr, d.tm_col, fact ? nullptr : d.tm_val, rs, d.tm_order, d.tm_n_long, g, ldo, dout,
                         GCNSA_EPI_NONE, nullptr, 0, M->tmp_b, ldo, SpmmBounds{n, n, d.tm_nnz}));
      } else {
        PROF_SPMM(M, spmm_cost(n, n, nnz, dout, !fact),
             launch_spmm(s, n, d.t_rowptr, d.t_col, fact ? nullptr : d.t_val, rs, d.t_order, d.t_n_long, g, ldo, dout,
                         GCNSA_EPI_NONE, nullptr, 0, M->tmp_b, ldo, SpmmBounds{n, n, nnz}));
      }
      PROF(M, 1, gemm_bytes(din, dout, n), 2.0 * n * dout * din,
           launch_gemm(s, M->o.gemm_mode, 1, 0, din, dout, n, hprev, ldi, M->tmp_b, ldo, gw, M->w_ld[l], 1, GCNSA_EPI_NONE,
                       nullptr, 0, M->ws, M->ws_bytes));
      bias_done = g_scaled = false;
      if (l > 0 && M->o.use_bias) {
        // G^{l-1}, its column sums (the bias gradient of layer l - 1) and, where the next transposed product wants
        // it, diag(dinv) G^{l-1} in place: one pass in the product's epilogue
        const bool want_scaled = fact && M->transform_first[l - 1];
        PROF(M, 1, gemm_bytes(n, din, dout) + 4.0 * n * din, 2.0 * n * dout * din,
             launch_gemm_mask_colsum(s, M->o.gemm_mode, 0, 1, n, din, dout, M->tmp_b, ldo, w, M->w_ld[l], M->tmp_a, ldi, hprev,
                                     ldi, want_scaled ? d.dinv : nullptr, M->gsum + M->b_off[l - 1], 1, M->sc, M->ws,
                                     M->ws_bytes));
        bias_done = true;
        g_scaled = want_scaled;
        g = M->tmp_a;
      } else if (l > 0) {
        PROF(M, 1, gemm_bytes(n, din, dout) + 4.0 * n * din, 2.0 * n * dout * din,
             launch_gemm(s, M->o.gemm_mode, 0, 1, n, din, dout, M->tmp_b, ldo, w, M->w_ld[l], M->tmp_a, ldi, 0, GCNSA_EPI_MASK,
                         hprev, ldi, M->ws, M->ws_bytes));
        g = M->tmp_a;
      }
    } else {
      bias_done = g_scaled = false;
      // dW += S^T G;  R = G W^T;  G^{l-1} = (A_hat^T R) .* [H^{l-1} > 0]
      PROF(M, 1, gemm_bytes(din, dout, n), 2.0 * n * dout * din,
           launch_gemm(s, M->o.gemm_mode, 1, 0, din, dout, n, l == 0 ? M->s0_used : M->S[l], ldi, g, ldo, gw, M->w_ld[l], 1,
                       GCNSA_EPI_NONE, nullptr, 0, M->ws, M->ws_bytes));
      if (l > 0) {
        PROF(M, 1, gemm_bytes(n, din, dout), 2.0 * n * dout * din,
             launch_gemm(s, M->o.gemm_mode, 0, 1, n, din, dout, g, ldo, w, M->w_ld[l], M->tmp_b, ldi, 0,
                         fact ? GCNSA_EPI_ROWSCALE : GCNSA_EPI_NONE, fact ? d.dinv : nullptr, 0, M->ws, M->ws_bytes));
        if (l == M->L - 1) {  // R = G W^T has the zero rows of G
          PROF_SPMM(M, spmm_cost(n, d.info.n_train, d.tm_nnz, din, !fact, true),
               launch_spmm(s, n, d.tm_rowptr, d.tm_col, fact ? nullptr : d.tm_val, rs, d.tm_order, d.tm_n_long, M->tmp_b, ldi, din,
                           GCNSA_EPI_MASK, hprev, ldi, M->tmp_a, ldi, SpmmBounds{n, n, d.tm_nnz}));
        } else {
          PROF_SPMM(M, spmm_cost(n, n, nnz, din, !fact, true),
               launch_spmm(s, n, d.t_rowptr, d.t_col, fact ? nullptr : d.t_val, rs, d.t_order, d.t_n_long, M->tmp_b, ldi, din,
                           GCNSA_EPI_MASK, hprev, ldi, M->tmp_a, ldi, SpmmBounds{n, n, nnz}));
        }
        g = M->tmp_a;
      }
    }
  }
  if (M->o.agg_mode == GCNSA_AGG_PARAM_AVG) {
    // this partition's own optimizer step from the aggregated parameters (Section 3.2), folded into the mean
    if (M->accumulated == 0)  // t -> t + 1 once per epoch
      PROF(M, 2, 0.0, 0.0, launch_adam_advance(s, M->adam_state, M->o.beta1, M->o.beta2));
    PROF(M, 2, 32.0 * M->count, 0.0,
         launch_adam_local_dev(s, M->count, M->theta, M->gsum, M->am_parts + (size_t)p * M->count,
                               M->av_parts + (size_t)p * M->count, M->theta_acc, M->accumulated == 0,
                               1.0f / (float)M->m, M->o.lr, M->o.beta1, M->o.beta2, M->o.eps, M->adam_state));
  }
  M->last_forward = -1;
  M->accumulated += 1;
  return GCNSA_OK;
}

int gcnsa_step(gcnsa_model* M) {
  if (!M) return fail(GCNSA_ERR_ARG, "model is NULL");
  if (M->accumulated != M->m) return fail(GCNSA_ERR_ORDER, "gcnsa_step needs one backward pass per partition");
  M->t += 1;
  if (M->o.agg_mode == GCNSA_AGG_PARAM_AVG) {
    CK(cudaMemcpyAsync(M->theta, M->theta_acc, (size_t)M->count * sizeof(float), cudaMemcpyDeviceToDevice, M->env.stream()));
    M->accumulated = 0;
    return GCNSA_OK;
  }
  PROF(M, 2, 0.0, 0.0, launch_adam_advance(M->env.e.stream, M->adam_state, M->o.beta1, M->o.beta2));  // t -> t + 1
  PROF(M, 2, 28.0 * M->count, 0.0,
       launch_adam_dev(M->env.e.stream, M->count, M->theta, M->gsum, M->am, M->av, 1.0f / (float)M->m, M->o.lr,
                       M->o.beta1, M->o.beta2, M->o.eps, M->adam_state));
  M->accumulated = 0;
  return GCNSA_OK;
}

static int epoch_body(gcnsa_model* M, const gcnsa_parts* P, float* loss_dev) {
  for (int32_t p = 0; p < P->m; ++p) {
    int rc = gcnsa_forward(M, P, p, nullptr);
    if (rc == GCNSA_OK) rc = gcnsa_backward(M, P, p);
    if (rc) return rc;
  }
  int rc = gcnsa_step(M);
  if (rc) return rc;
  if (loss_dev) CKL(launch_mean(M->env.e.stream, M->loss_parts, M->m, loss_dev));
  return GCNSA_OK;
}

int gcnsa_epoch(gcnsa_model* M, const gcnsa_parts* P, float* loss_dev) {
  if (!M || !P) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (M->accumulated != 0) return fail(GCNSA_ERR_ORDER, "gcnsa_epoch needs an empty gradient sum");
  cudaStream_t s = M->env.stream();
  const bool want_graph = M->o.epoch_graph && !M->graph_off && !M->prof_on && s != nullptr;
  if (!want_graph) return epoch_body(M, P, loss_dev);
  if (M->o.cache_ax && P->uid == M->ax_uid && P->m == M->m)  // outside the recording: a replay only reads the cached products
    for (int32_t p = 0; p < P->m; ++p) {
      int rc = ensure_ax(M, P, p);
      if (rc) return rc;
    }
  if (M->graph_exec && (M->graph_parts_uid != P->uid || M->graph_loss != (const void*)loss_dev)) {
    cudaGraphExecDestroy(M->graph_exec);
    M->graph_exec = nullptr;
  }
  if (!M->graph_exec) {
    // record one epoch; the launches only describe work, nothing runs until the graph is launched
    const int64_t t0 = M->t;
    const int64_t launches0 = gcnsa_launch_count();
    cudaGraph_t graph = nullptr;
    int rc = GCNSA_OK;
    if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      M->graph_off = true;
      return epoch_body(M, P, loss_dev);
    }
    rc = epoch_body(M, P, loss_dev);
    cudaError_t e = cudaStreamEndCapture(s, &graph);
    M->t = t0;  // the host's copy of the step count advances when the graph runs
    M->accumulated = 0;
    M->last_forward = -1;
    const int recorded = (int)(gcnsa_launch_count() - launches0);
    note_launch(-recorded);  // recorded, not launched
    if (rc != GCNSA_OK || e != cudaSuccess || !graph ||
        cudaGraphInstantiate(&M->graph_exec, graph, 0) != cudaSuccess) {
      if (graph) cudaGraphDestroy(graph);
      cudaGetLastError();
      M->graph_exec = nullptr;
      M->graph_off = true;  // this stream or driver cannot record the epoch: plain launches from now on
      return epoch_body(M, P, loss_dev);
    }
    cudaGraphDestroy(graph);
    M->graph_parts_uid = P->uid;
    M->graph_loss = (const void*)loss_dev;
    M->graph_kernels = recorded;
  }
  CK(cudaGraphLaunch(M->graph_exec, s));
  note_launch(M->graph_kernels);
  M->t += 1;
  M->last_n = P->parts[P->m - 1].info.n;
  return GCNSA_OK;
}

int gcnsa_epoch_host(gcnsa_model* M, gcnsa_parts* P, const float* const* x_host, float* loss_host) {
  if (!M || !P || !x_host || !loss_host) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (M->accumulated != 0) return fail(GCNSA_ERR_ORDER, "gcnsa_epoch_host needs an empty gradient sum");
  for (int32_t p = 0; p < P->m; ++p)
    if (!x_host[p]) return fail(GCNSA_ERR_ARG, "x_host[p] is NULL");
  cudaStream_t s = M->env.stream();
  if (!P->copy_stream) {  // first use: copy stream, events, two staging buffers
    CK(cudaStreamCreateWithFlags(&P->copy_stream, cudaStreamNonBlocking));
    P->ready.resize((size_t)P->m);
    P->consumed.resize((size_t)P->m);
    for (int32_t p = 0; p < P->m; ++p) {
      CK(cudaEventCreateWithFlags(&P->ready[p], cudaEventDisableTiming));
      CK(cudaEventCreateWithFlags(&P->consumed[p], cudaEventDisableTiming));
      CK(cudaEventRecord(P->consumed[p], s));
    }
  }
  for (int b = 0; b < 2; ++b) {  // (a call that ran out of memory here leaves what it got for the next one)
    if (P->staging[b]) continue;
    P->staging[b] = (float*)P->dalloc((size_t)std::max<int64_t>(P->n_max, 1) * (size_t)P->f * sizeof(float));
    if (!P->staging[b]) return fail(GCNSA_ERR_OOM, "device allocation failed");
  }
  // uploads run on their own stream, one partition ahead of the compute stream:
  // dense host rows -> staging buffer -> padded device rows
  for (int32_t p = 0; p < P->m; ++p) {
    DevPart& d = P->parts[p];
    CK(cudaStreamWaitEvent(P->copy_stream, P->consumed[p], 0));  // the previous reader of X_p has finished
    float* st = P->staging[p & 1];
    CK(cudaMemcpyAsync(st, x_host[p], (size_t)d.info.n * (size_t)P->f * sizeof(float), cudaMemcpyHostToDevice,
                       P->copy_stream));
    CKL(launch_repitch(P->copy_stream, d.info.n, P->f, st, d.x, P->ldx));
    P->x_version[p] += 1;
    CK(cudaEventRecord(P->ready[p], P->copy_stream));
  }
  for (int32_t p = 0; p < P->m; ++p) {
    CK(cudaStreamWaitEvent(s, P->ready[p], 0));
    int rc = gcnsa_forward(M, P, p, nullptr);
    if (rc == GCNSA_OK) rc = gcnsa_backward(M, P, p);
    if (rc) return rc;
    CK(cudaEventRecord(P->consumed[p], s));
  }
  int rc = gcnsa_step(M);
  if (rc) return rc;
  float* mean_dev = M->loss_parts + M->m;  // slot after the M partition losses
  CKL(launch_mean(M->env.e.stream, M->loss_parts, M->m, mean_dev));
  CK(cudaMemcpyAsync(loss_host, mean_dev, sizeof(float), cudaMemcpyDeviceToHost, M->env.stream()));
  CK(cudaStreamSynchronize(M->env.stream()));
  return GCNSA_OK;
}

}  // extern "C"

// ------------------------------------------------------- get / set / ops ---
extern "C" {

static float* param_base(const gcnsa_model* M, int32_t what, bool* is_w) {
  switch (what) {
    case GCNSA_GET_W: *is_w = true; return M->theta;
    case GCNSA_GET_B: *is_w = false; return M->theta;
    case GCNSA_GET_GRAD_W: *is_w = true; return M->gsum;
    case GCNSA_GET_GRAD_B: *is_w = false; return M->gsum;
    case GCNSA_GET_ADAM_M_W: *is_w = true; return M->am_parts ? M->am_parts + (size_t)M->state_p * M->count : M->am;
    case GCNSA_GET_ADAM_M_B: *is_w = false; return M->am_parts ? M->am_parts + (size_t)M->state_p * M->count : M->am;
    case GCNSA_GET_ADAM_V_W: *is_w = true; return M->av_parts ? M->av_parts + (size_t)M->state_p * M->count : M->av;
    case GCNSA_GET_ADAM_V_B: *is_w = false; return M->av_parts ? M->av_parts + (size_t)M->state_p * M->count : M->av;
    default: return nullptr;
  }
}

int gcnsa_model_get(const gcnsa_model* M, int32_t what, int32_t layer, void* host_dst, size_t bytes) {
  if (!M || !host_dst) return fail(GCNSA_ERR_ARG, "NULL argument");
  bool is_w = false;
  if (float* base = param_base(M, what, &is_w)) {
    if (layer < 0 || layer >= M->L) return fail(GCNSA_ERR_ARG, "layer out of range");
    return copy_param(M, base, layer, is_w, host_dst, bytes, true);
  }
  const float* src = nullptr;
  int64_t cols = 0;
  if (what == GCNSA_GET_ACT) {
    if (layer < 1 || layer > M->L) return fail(GCNSA_ERR_ARG, "layer out of range");
    src = M->H[layer];
    cols = M->o.dims[layer];
  } else if (what == GCNSA_GET_DLOGITS) {
    src = M->dlogits;
    cols = M->o.dims[M->L];
  } else {
    return fail(GCNSA_ERR_ARG, "unknown tensor id");
  }
  if (bytes != (size_t)(M->last_n * cols) * sizeof(float)) return fail(GCNSA_ERR_ARG, "byte count does not match the tensor");
  if (M->last_n > 0)
    CK(cudaMemcpy2DAsync(host_dst, (size_t)cols * sizeof(float), src, (size_t)GCNSA_LD(cols) * sizeof(float),
                         (size_t)cols * sizeof(float), (size_t)M->last_n, cudaMemcpyDeviceToHost, M->env.stream()));
  CK(cudaStreamSynchronize(M->env.stream()));
  return GCNSA_OK;
}

int gcnsa_model_set(gcnsa_model* M, int32_t what, int32_t layer, const void* host_src, size_t bytes) {
  if (!M || !host_src) return fail(GCNSA_ERR_ARG, "NULL argument");
  bool is_w = false;
  float* base = param_base(M, what, &is_w);
  if (!base) return fail(GCNSA_ERR_ARG, "tensor cannot be set");
  if (layer < 0 || layer >= M->L) return fail(GCNSA_ERR_ARG, "layer out of range");
  return copy_param(M, base, layer, is_w, (void*)host_src, bytes, false);
}

int gcnsa_model_profile(gcnsa_model* M, int32_t enable) {
  if (!M) return fail(GCNSA_ERR_ARG, "model is NULL");
  CK(cudaStreamSynchronize(M->env.stream()));
  M->prof_on = enable != 0;
  M->recs.clear();
  return GCNSA_OK;
}

int gcnsa_model_profile_read(gcnsa_model* M, gcnsa_profile* out) {
  if (!M || !out) return fail(GCNSA_ERR_ARG, "NULL argument");
  std::memset(out, 0, sizeof(*out));
  CK(cudaStreamSynchronize(M->env.stream()));
  for (size_t i = 0; i < M->recs.size(); ++i) {
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, M->ev[2 * i], M->ev[2 * i + 1]));
    const auto& r = M->recs[i];
    out->ms[r.cat] += ms;
    out->launches[r.cat] += r.launches;
    out->alg_bytes[r.cat] += r.bytes;
    out->l1_bytes[r.cat] += r.l1;
    out->alg_bytes_val[r.cat] += r.bytes_val;
    out->flops[r.cat] += r.flops;
  }
  M->recs.clear();
  return GCNSA_OK;
}

int gcnsa_evaluate(gcnsa_model* M, const gcnsa_parts* P, int32_t p, const uint8_t* mask_host, int64_t* correct_host,
                   int64_t* total_host, int32_t* pred_host) {
  if (!M || !P || !correct_host || !total_host || p < 0 || p >= P->m)
    return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  if (M->accumulated != 0 || M->last_forward >= 0)
    return fail(GCNSA_ERR_ORDER, "gcnsa_evaluate between a forward pass and gcnsa_step");
  if (!M->ev_pred) M->ev_pred = (int32_t*)M->dalloc((size_t)M->n_max * sizeof(int32_t));
  if (!M->ev_hits) M->ev_hits = (int32_t*)M->dalloc(4096 * sizeof(int32_t));
  if (!M->ev_mask) M->ev_mask = (uint8_t*)M->dalloc((size_t)M->n_max);
  if (!M->ev_pred || !M->ev_hits || !M->ev_mask) return fail(GCNSA_ERR_OOM, "device allocation failed");
  M->all_rows_once = true;
  int rc = gcnsa_forward(M, P, p, nullptr);   // also checks that the model fits these partitions
  M->all_rows_once = false;
  if (rc) return rc;
  M->last_forward = -1;                       // an evaluation pass is not followed by a backward pass
  const DevPart& d = P->parts[p];
  const int64_t n = d.info.n;
  cudaStream_t s = M->env.stream();
  if (mask_host && n > 0) CK(cudaMemcpyAsync(M->ev_mask, mask_host, (size_t)n, cudaMemcpyHostToDevice, s));
  int blocks = 0;
  CKL(launch_argmax_hits(s, n, P->c, M->H[M->L], GCNSA_LD(P->c), d.y, mask_host ? M->ev_mask : nullptr, M->ev_pred,
                         M->ev_hits, &blocks));
  std::vector<int32_t> hits((size_t)std::max(blocks, 1), 0);
  if (n > 0) CK(cudaMemcpyAsync(hits.data(), M->ev_hits, (size_t)blocks * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  if (pred_host && n > 0) CK(cudaMemcpyAsync(pred_host, M->ev_pred, (size_t)n * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  int64_t correct = 0, total = 0;
  for (int b = 0; b < blocks && n > 0; ++b) correct += hits[b];
  for (int64_t i = 0; i < n; ++i) total += mask_host ? (mask_host[i] != 0) : 1;
  *correct_host = correct;
  *total_host = total;
  return GCNSA_OK;
}

int gcnsa_model_copy_params(gcnsa_model* dst, const gcnsa_model* src) {
  if (!dst || !src) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (dst->L != src->L || dst->count != src->count) return fail(GCNSA_ERR_ARG, "models have different dims");
  for (int l = 0; l <= dst->L; ++l)
    if (dst->o.dims[l] != src->o.dims[l]) return fail(GCNSA_ERR_ARG, "models have different dims");
  CK(cudaStreamSynchronize(src->env.stream()));
  CK(cudaMemcpyAsync(dst->theta, src->theta, (size_t)dst->count * sizeof(float), cudaMemcpyDeviceToDevice,
                     dst->env.stream()));
  return GCNSA_OK;
}

int gcnsa_model_select_partition(gcnsa_model* M, int32_t p) {
  if (!M || p < 0 || p >= M->m) return fail(GCNSA_ERR_ARG, "NULL model or partition index out of range");
  M->state_p = p;
  return GCNSA_OK;
}

int gcnsa_model_get_t(const gcnsa_model* M, int64_t* t_out) {
  if (!M || !t_out) return fail(GCNSA_ERR_ARG, "NULL argument");
  *t_out = M->t;
  return GCNSA_OK;
}
int gcnsa_model_set_t(gcnsa_model* M, int64_t t) {
  if (!M || t < 0) return fail(GCNSA_ERR_ARG, "NULL model or negative step count");
  M->t = t;
  // the kernels read the count from device memory; the bias corrections are recomputed at the next step
  const double state[4] = {(double)t, 0.0, 0.0, 0.0};
  CK(cudaMemcpyAsync(M->adam_state, state, sizeof(state), cudaMemcpyHostToDevice, M->env.stream()));
  CK(cudaStreamSynchronize(M->env.stream()));
  return GCNSA_OK;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

int gcnsa_op_spmm(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                  const int32_t* order, int64_t n_long, const float* x, int64_t ldx, int32_t f, int32_t epi, const float* aux,
                  int64_t ldaux, float* y, int64_t ldy) {
  if (n_rows < 0 || f < 0 || n_rows >= INT32_MAX) return fail(GCNSA_ERR_ARG, "negative or oversized dimension");
  if (n_rows == 0 || f == 0) return GCNSA_OK;
  if (!rowptr || !col || !val || !x || !y) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (ldx % 4 || ldy % 4 || ldx < f || ldy < f || !aligned16(x) || !aligned16(y))
    return fail(GCNSA_ERR_ARG, "x and y need 16-byte aligned bases and leading dimensions that are multiples of 4");
  if (epi < GCNSA_EPI_NONE || epi > GCNSA_EPI_MASK) return fail(GCNSA_ERR_ARG, "unknown epilogue");
  if (epi == GCNSA_EPI_MASK && (!aux || ldaux % 4 || ldaux < f || !aligned16(aux)))
    return fail(GCNSA_ERR_ARG, "mask needs a 16-byte aligned base and a leading dimension that is a multiple of 4");
  if (epi == GCNSA_EPI_BIAS && !aux) return fail(GCNSA_ERR_ARG, "bias is NULL");
  if (n_long < 0 || n_long > n_rows) return fail(GCNSA_ERR_ARG, "n_long out of range");
  CKL(launch_spmm(stream, n_rows, rowptr, col, val, nullptr, order, n_long, x, ldx, f, epi, aux, ldaux, y, ldy,
                  SpmmBounds{n_rows, -1, -1}));
  return GCNSA_OK;
}

int gcnsa_op_spmm_pattern(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* row_scale,
                          const int32_t* order, int64_t n_long, const float* x, int64_t ldx, int32_t f, int32_t epi,
                          const float* aux, int64_t ldaux, float* y, int64_t ldy) {
  if (n_rows < 0 || f < 0 || n_rows >= INT32_MAX) return fail(GCNSA_ERR_ARG, "negative or oversized dimension");
  if (n_rows == 0 || f == 0) return GCNSA_OK;
  if (!rowptr || !col || !x || !y) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (ldx % 4 || ldy % 4 || ldx < f || ldy < f || !aligned16(x) || !aligned16(y))
    return fail(GCNSA_ERR_ARG, "x and y need 16-byte aligned bases and leading dimensions that are multiples of 4");
  if (epi < GCNSA_EPI_NONE || epi > GCNSA_EPI_MASK) return fail(GCNSA_ERR_ARG, "unknown epilogue");
  if (epi == GCNSA_EPI_MASK && (!aux || ldaux % 4 || ldaux < f || !aligned16(aux)))
    return fail(GCNSA_ERR_ARG, "mask needs a 16-byte aligned base and a leading dimension that is a multiple of 4");
  if (epi == GCNSA_EPI_BIAS && !aux) return fail(GCNSA_ERR_ARG, "bias is NULL");
  if (n_long < 0 || n_long > n_rows) return fail(GCNSA_ERR_ARG, "n_long out of range");
  CKL(launch_spmm(stream, n_rows, rowptr, col, nullptr, row_scale, order, n_long, x, ldx, f, epi, aux, ldaux, y, ldy,
                  SpmmBounds{n_rows, -1, -1}));
  return GCNSA_OK;
}

size_t gcnsa_op_gemm_workspace(int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k) {
  if (m <= 0 || n <= 0 || k <= 0) return 0;
  return gemm_workspace(mode, ta, tb, m, n, k);
}

int gcnsa_tc_status(int32_t* status_host) {
  if (!status_host) return fail(GCNSA_ERR_ARG, "NULL argument");
  CK(cudaDeviceSynchronize());
  int v = 0;
  CKL(tc_status(&v));
  *status_host = v;
  return GCNSA_OK;
}

int gcnsa_debug_status(int32_t* enabled_host, int32_t* code_host, int64_t* value_host) {
  if (!enabled_host || !code_host || !value_host) return fail(GCNSA_ERR_ARG, "NULL argument");
#ifdef GCNSA_DEBUG
  *enabled_host = 1;
#else
  *enabled_host = 0;
#endif
  *code_host = 0;
  *value_host = 0;
  CK(cudaDeviceSynchronize());
  unsigned long long w[2] = {0ull, 0ull};
  CKL(debug_word_spmm(&w[0], true));
  CKL(debug_word_build(&w[1], true));
  const unsigned long long first = w[0] ? w[0] : w[1];
  *code_host = (int32_t)(first >> 56);
  *value_host = (int64_t)(first & 0x00ffffffffffffffull);
  return GCNSA_OK;
}

int gcnsa_tc_clear(void) {
  CK(cudaDeviceSynchronize());
  CKL(tc_clear());
  return GCNSA_OK;
}

int gcnsa_op_gemm(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a,
                  int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi,
                  const float* aux, int64_t ldaux, void* workspace, size_t workspace_bytes) {
  if (m < 0 || n < 0 || k < 0) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (mode != GCNSA_GEMM_FP32 && mode != GCNSA_GEMM_TF32X3 && mode != GCNSA_GEMM_TF32)
    return fail(GCNSA_ERR_ARG, "unknown gemm mode");
  if (m == 0 || n == 0) return GCNSA_OK;
  if (!c || (k > 0 && (!a || !b))) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (lda < (ta ? m : k) || ldb < (tb ? k : n) || ldc < n) return fail(GCNSA_ERR_ARG, "leading dimension too small");
  if (epi < GCNSA_EPI_NONE || epi > GCNSA_EPI_ROWSCALE) return fail(GCNSA_ERR_ARG, "unknown epilogue");
  if ((epi == GCNSA_EPI_MASK || epi == GCNSA_EPI_BIAS || epi == GCNSA_EPI_ROWSCALE) && !aux)
    return fail(GCNSA_ERR_ARG, "aux is NULL");
  CKL(launch_gemm(stream, mode, ta, tb, m, n, k, a, lda, b, ldb, c, ldc, accumulate, epi, aux, ldaux, workspace,
                  workspace_bytes));
  return GCNSA_OK;
}

size_t gcnsa_op_gemm_mask_colsum_scratch(int64_t m, int32_t n) {
  return (gemm_colsum_scratch(m < 0 ? 0 : m, n < 0 ? 0 : n) + 255) / 256 * 256;
}

int gcnsa_op_gemm_mask_colsum(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k,
                              const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc,
                              const float* mask, int64_t ldmask, const float* row_scale, float* out,
                              int32_t accumulate, void* scratch, size_t scratch_bytes, void* workspace,
                              size_t workspace_bytes) {
  if (m < 0 || n < 0 || k < 0 || n >= (1LL << 31)) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (mode != GCNSA_GEMM_FP32 && mode != GCNSA_GEMM_TF32X3 && mode != GCNSA_GEMM_TF32)
    return fail(GCNSA_ERR_ARG, "unknown gemm mode");
  if (n > 0 && !out) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (m == 0 || n == 0) {
    if (n > 0 && !accumulate) CK(cudaMemsetAsync(out, 0, (size_t)n * sizeof(float), (cudaStream_t)stream));
    return GCNSA_OK;
  }
  if (!c || !mask || (k > 0 && (!a || !b))) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (lda < (ta ? m : k) || ldb < (tb ? k : n) || ldc < n || ldmask < n) return fail(GCNSA_ERR_ARG, "leading dimension too small");
  if (!scratch || ((uintptr_t)scratch & 255) || scratch_bytes < gemm_colsum_scratch(m, (int32_t)n))
    return fail(GCNSA_ERR_ARG, "scratch missing, unaligned or too small");
  CKL(launch_gemm_mask_colsum(stream, mode, ta, tb, m, n, k, a, lda, b, ldb, c, ldc, mask, ldmask, row_scale, out, accumulate,
                              scratch, workspace, workspace_bytes));
  return GCNSA_OK;
}

static int probe_sms(int* sms) {
  int dev = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev));
  return GCNSA_OK;
}

int gcnsa_op_gather_probe_warps(int32_t* warps_out) {
  if (!warps_out) return fail(GCNSA_ERR_ARG, "NULL pointer");
  int sms = 0;
  int rc = probe_sms(&sms);
  if (rc) return rc;
  *warps_out = gather_probe_warps(sms);
  return GCNSA_OK;
}

int gcnsa_op_gather_probe(void* stream, const float* x, int64_t ldx, int64_t n_rows, int32_t window_rows,
                          int32_t hit_every, int32_t rounds, float* out, size_t out_bytes) {
  if (!x || !out) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (ldx < 128 || (ldx % 4) || ((uintptr_t)x & 15) || ((uintptr_t)out & 15))
    return fail(GCNSA_ERR_ARG, "rows of at least 128 floats, 16-byte aligned");
  if (n_rows < 1 || n_rows >= (1LL << 31) || window_rows < 1 || window_rows > n_rows || hit_every < 0 || rounds < 0)
    return fail(GCNSA_ERR_ARG, "row counts, hit_every or rounds out of range");
  int sms = 0;
  int rc = probe_sms(&sms);
  if (rc) return rc;
  if (out_bytes < (size_t)gather_probe_warps(sms) * 128 * sizeof(float)) return fail(GCNSA_ERR_ARG, "out too small");
  CKL(launch_gather_probe(stream, x, ldx, n_rows, window_rows, hit_every, rounds, out, sms));
  return GCNSA_OK;
}

size_t gcnsa_op_softmax_ce_scratch(int64_t n) { return softmax_ce_scratch(n < 0 ? 0 : n); }

int gcnsa_op_softmax_ce(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                        const uint8_t* mask, int64_t n_train, float* loss_dev, float* grad, int64_t ldg, void* scratch,
                        size_t scratch_bytes) {
  if (n < 0 || c < 1 || n_train < 0) return fail(GCNSA_ERR_ARG, "negative dimension or c < 1");
  if (n > 0 && (!logits || !y || !mask || !grad)) return fail(GCNSA_ERR_ARG, "NULL pointer");
  if (ld < c || ldg < c) return fail(GCNSA_ERR_ARG, "leading dimension too small");
  if (!scratch || scratch_bytes < softmax_ce_scratch(n)) return fail(GCNSA_ERR_ARG, "scratch too small");
  CKL(launch_softmax_ce(stream, n, c, logits, ld, y, mask, n_train, loss_dev, grad, ldg, scratch));
  return GCNSA_OK;
}

size_t gcnsa_op_colsum_scratch(int64_t n, int32_t f) { return colsum_scratch(n < 0 ? 0 : n, f < 0 ? 0 : f); }

int gcnsa_op_colsum(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                    void* scratch, size_t scratch_bytes) {
  if (n < 0 || f < 0) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (f == 0) return GCNSA_OK;
  if (!out || (n > 0 && !g) || ldg < f) return fail(GCNSA_ERR_ARG, "NULL pointer or leading dimension too small");
  if (!scratch || scratch_bytes < colsum_scratch(n, f)) return fail(GCNSA_ERR_ARG, "scratch too small");
  CKL(launch_colsum(stream, n, f, g, ldg, out, accumulate, scratch));
  return GCNSA_OK;
}

int gcnsa_op_colsum_scaled(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                           void* scratch, size_t scratch_bytes, const float* row_scale, float* scaled, int64_t lds) {
  if (n < 0 || f < 0) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (f == 0) return GCNSA_OK;
  if (!out || (n > 0 && !g) || ldg < f) return fail(GCNSA_ERR_ARG, "NULL pointer or leading dimension too small");
  if (!scratch || scratch_bytes < colsum_scratch(n, f)) return fail(GCNSA_ERR_ARG, "scratch too small");
  if (!row_scale || !scaled) return fail(GCNSA_ERR_ARG, "row_scale or scaled is NULL");
  if (lds % 4 || ldg % 4 || lds < (f + 3) / 4 * 4 || ldg < (f + 3) / 4 * 4 || !aligned16(scaled) || !aligned16(g))
    return fail(GCNSA_ERR_ARG, "g and scaled need 16-byte aligned bases and leading dimensions that are multiples of 4");
  CKL(launch_colsum_scaled(stream, n, f, g, ldg, out, accumulate, scratch, row_scale, scaled, lds));
  return GCNSA_OK;
}

int gcnsa_op_adam(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m, float lr,
                  float beta1, float beta2, float eps, int64_t t) {
  if (count < 0 || t < 1) return fail(GCNSA_ERR_ARG, "negative count or t < 1");
  if (count > 0 && (!theta || !gsum || !m || !v)) return fail(GCNSA_ERR_ARG, "NULL pointer");
  CKL(launch_adam(stream, count, theta, gsum, m, v, inv_m, lr, beta1, beta2, eps, t));
  return GCNSA_OK;
}

int gcnsa_op_normalize(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const int32_t* deg,
                       float* val) {
  if (n_rows < 0) return fail(GCNSA_ERR_ARG, "negative dimension");
  if (n_rows > 0 && (!rowptr || !col || !deg || !val)) return fail(GCNSA_ERR_ARG, "NULL pointer");
  CKL(launch_normalize(stream, n_rows, rowptr, col, deg, val));
  return GCNSA_OK;
}

}  // extern "C"

// ------------------------------------------------------------------- plan ---
struct gcnsa_plan {
  HostBuild hb;
  int32_t m = 0;
};

extern "C" {

int gcnsa_plan_create(const gcnsa_graph* g, const gcnsa_part_opts* opts, gcnsa_plan** out) {
  if (!out) return fail(GCNSA_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (!g || !opts) return fail(GCNSA_ERR_ARG, "NULL argument");
  gcnsa_plan* pl = new (std::nothrow) gcnsa_plan();
  if (!pl) return fail(GCNSA_ERR_OOM, "host allocation failed");
  int rc = build_host(g, opts, &pl->hb);
  if (rc) {
    delete pl;
    return rc;
  }
  pl->m = opts->m;
  *out = pl;
  return GCNSA_OK;
}

int gcnsa_plan_info(const gcnsa_plan* plan, int32_t p, gcnsa_part_info* out) {
  if (!plan || !out || p < 0 || p >= plan->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const HostPart& hp = plan->hb.parts[p];
  out->n_owned = hp.n_owned; out->n_halo = hp.n_halo; out->n = hp.n; out->nnz = hp.nnz; out->nts = hp.nts;
  out->n_train = hp.n_train; out->max_depth = hp.max_depth;
  return GCNSA_OK;
}

int gcnsa_plan_assignment(const gcnsa_plan* plan, int32_t* part_host) {
  if (!plan || !part_host) return fail(GCNSA_ERR_ARG, "NULL argument");
  std::memcpy(part_host, plan->hb.part.data(), plan->hb.part.size() * sizeof(int32_t));
  return GCNSA_OK;
}

int gcnsa_plan_export(const gcnsa_plan* plan, int32_t p, const gcnsa_part_host* dst) {
  if (!plan || !dst || p < 0 || p >= plan->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const HostPart& hp = plan->hb.parts[p];
  if (dst->rowptr) std::memcpy(dst->rowptr, hp.rowptr.data(), hp.rowptr.size() * sizeof(int32_t));
  if (dst->col) std::memcpy(dst->col, hp.col.data(), hp.col.size() * sizeof(int32_t));
  if (dst->t_rowptr) std::memcpy(dst->t_rowptr, hp.t_rowptr.data(), hp.t_rowptr.size() * sizeof(int32_t));
  if (dst->t_col) std::memcpy(dst->t_col, hp.t_col.data(), hp.t_col.size() * sizeof(int32_t));
  if (dst->members) std::memcpy(dst->members, hp.members.data(), hp.members.size() * sizeof(int64_t));
  if (dst->depth) std::memcpy(dst->depth, hp.depth.data(), hp.depth.size() * sizeof(int32_t));
  return GCNSA_OK;
}

int gcnsa_plan_export_schedule(const gcnsa_plan* plan, int32_t p, gcnsa_part_schedule_info* info,
                               const gcnsa_part_schedule_host* dst) {
  if (!plan || p < 0 || p >= plan->m) return fail(GCNSA_ERR_ARG, "bad partition index or NULL");
  const HostPart& hp = plan->hb.parts[p];
  if (info) {
    info->n_long = hp.n_long; info->t_n_long = hp.t_n_long; info->m_n_long = hp.m_n_long; info->tm_n_long = hp.tm_n_long;
    info->m_nnz = hp.m_nnz; info->tm_nnz = (int64_t)hp.tm_col.size();
  }
  if (!dst) return GCNSA_OK;
  auto put = [](int32_t* to, const std::vector<int32_t>& from) {
    if (to && !from.empty()) std::memcpy(to, from.data(), from.size() * sizeof(int32_t));
  };
  put(dst->order, hp.order); put(dst->t_order, hp.t_order); put(dst->m_order, hp.m_order);
  put(dst->tm_rowptr, hp.tm_rowptr); put(dst->tm_col, hp.tm_col); put(dst->tm_order, hp.tm_order);
  return GCNSA_OK;  // mask and y are gathered on the device only
}

int gcnsa_plan_destroy(gcnsa_plan* plan) {
  delete plan;
  return GCNSA_OK;
}

}  // extern "C"
