// Internal declarations shared by the translation units of libgcnsa.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "debug_check.h"
#include "gcnsa.h"

namespace gcnsa {

// A row is handed to a whole thread block instead of a warp when one warp's serial chain over it would be a
// large part of the launch: at least kLongRow non-zeros and more than 1/8192 of the matrix (about half of what
// each of the ~4 700 resident warps gets).  Measured on the paper-scale graph: 16 partitions 2.2x faster with
// long rows split, 5 partitions 3 % slower if rows of 1 024 are split too early.
constexpr int kLongRow = 1024;
inline int64_t long_row_threshold(int64_t nnz) { return nnz / 8192 > kLongRow ? nnz / 8192 : kLongRow; }

#ifdef __CUDACC__
#define GCNSA_HD __host__ __device__
#else
#define GCNSA_HD
#endif

// Processing order of the rows of a product: hub rows (at least `thr` entries) first; then the other rows window by
// window, a window being `window` consecutive rows of the matrix; inside a window by descending length class, rows of
// one class in index order.  A class holds the lengths that agree in their five leading bits (3-6 % apart; lengths
// below 32 are a class each).  The warps of a block then finish together, as with a strict length order, and they
// work on neighbouring rows, which in a graph with community-ordered ids gather overlapping sets of source rows at
// the same time (L1 hits: 458 -> 434 us at F' = 128 on the paper-scale partition; blocks of neighbouring rows without
// the length classes were 1.3-1.9 x slower).  The windows bound the set of source rows that is live at any time:
// without them the rows in flight are spread over the whole partition, and when the gathered matrix exceeds L2
// (2.45 M-vertex graph, width 256: 276 MB) its rows are fetched from HBM several times over.
constexpr int64_t kOrderWindow = 8192;     // rows per window unless the caller says otherwise
constexpr int64_t kOrderWindowMin = 256;   // keeps (windows + 1) x classes inside 32 bits for any int32 row count
GCNSA_HD inline int32_t length_class(int64_t len) {
  if (len < 32) return (int32_t)(len < 0 ? 0 : len);
  int e = 5;
  while ((len >> (e + 1)) != 0) ++e;  // e = floor(log2(len))
  return 32 + (e - 5) * 16 + (int32_t)((len >> (e - 4)) & 15);
}
// sort key (ascending = processing order) of row `row` with `len` entries in a matrix of `n_rows` rows;
// window <= 0: one window over all rows
GCNSA_HD inline uint32_t order_key(int64_t len, int64_t thr, int64_t n_rows, int64_t row, int64_t window) {
  const int32_t cmax = length_class(n_rows + 1);
  const int32_t c = length_class(len);
  if (len >= thr) return (uint32_t)(cmax - c);
  const int64_t w = window > 0 ? row / window : 0;
  return (uint32_t)((w + 1) * (int64_t)(cmax + 1) + (cmax - c));
}
GCNSA_HD inline int order_key_bits(int64_t n_rows, int64_t window) {
  const int64_t n_win = window > 0 ? (n_rows + window - 1) / window : 1;
  const uint64_t top = (uint64_t)(n_win + 1) * (uint64_t)(length_class(n_rows + 1) + 1);
  int b = 1;
  while ((top >> b) != 0) ++b;
  return b;
}
// Rows per window for an order_window option and a matrix of n_rows rows (0 = one window over all rows).
// Option 0 lets the row count decide: windows pay when the gathered matrix exceeds L2 (2.45 M-vertex graph, 270 K
// rows per partition: 21.9 -> 23.8 epochs/s) and cost when it is L2-resident, where they concentrate all SMs on the
// few megabytes of one community (233 K-vertex graph, 51 K rows per partition: 140 -> 117 epochs/s).  The widths of
// the model are not known when partitions are built, so the rule goes by rows: from kOrderWindowFrom rows on, a
// matrix of 256 floats per row is as large as L2.
constexpr int64_t kOrderWindowFrom = 131072;
inline int64_t order_window_rows(int32_t opt, int64_t n_rows) {
  if (opt == 0) return n_rows >= kOrderWindowFrom ? kOrderWindow : 0;
  return opt < 0 ? 0 : (int64_t)opt;
}

// ---- errors -----------------------------------------------------------------
int fail(int code, const std::string& detail);  // records the thread-local text, returns code
void note_launch(int n = 1);
// one dense product handed to launch_gemm in GCNSA_GEMM_TF32X3 mode: it ran on the tensor-core kernel, or on the
// fp32 FMA kernel because the tensor-core path could not take it
void note_gemm_path(bool tensor_core);

// ---- host-side result of the partition builder --------------------------------
struct HostPart {
  int64_t n_owned = 0, n_halo = 0, n = 0, nnz = 0, nts = 0, n_train = 0;
  int32_t max_depth = 0;
  std::vector<int64_t> members;  // local -> global
  std::vector<int32_t> depth;    // per other partition
  std::vector<int32_t> rowptr, col, t_rowptr, t_col;
  // transposed CSR restricted to the columns that carry loss: the gradient of the loss w.r.t. the logits has
  // zero rows elsewhere, so the last layer's transposed product only needs these non-zeros
  std::vector<int32_t> tm_rowptr, tm_col, tm_order;
  int64_t tm_n_long = 0;
  std::vector<int32_t> m_order;  // the rows that carry loss, by descending length
  int64_t m_n_long = 0, m_nnz = 0;  // m_nnz: non-zeros in those rows
  std::vector<int32_t> order;    // rows by descending length (processing order)
  std::vector<int32_t> t_order;
  int64_t n_long = 0, t_n_long = 0;  // long rows (see long_row_threshold): the head of order / t_order
};

struct HostBuild {
  std::vector<int32_t> part;
  std::vector<HostPart> parts;
};

// Partition assignment + Algorithm 1 + induced graphs (structure only).
int build_host(const gcnsa_graph* g, const gcnsa_part_opts* o, HostBuild* out);

// 64-bit selection key (SplitMix64 finalizer applied word by word).
uint64_t selection_key(uint64_t seed, uint64_t w0, uint64_t w1, uint64_t w2, uint64_t w3, uint64_t v);

// ---- kernel launchers (all enqueue on `stream`, return a cudaError_t as int) ---
// val == NULL: every stored entry counts as 1; row_scale (nullable): row i of the sum is multiplied by row_scale[i]
// before the epilogue
// bounds: what the caller knows about the operands, checked by the kernels of the GCNSA_DEBUG build only
int launch_spmm(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                const float* row_scale, const int32_t* order, int64_t n_long, const float* x, int64_t ldx, int32_t f, int32_t epi, const float* aux,
                int64_t ldaux, float* y, int64_t ldy, const SpmmBounds& bounds = SpmmBounds());
int launch_gemm(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a,
                int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi,
                const float* aux, int64_t ldaux, void* workspace, size_t workspace_bytes);
size_t gemm_workspace(int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k);
// tensor-core path (3xTF32); returns -1 when the call has to fall back to the fp32 FMA kernel
// terms: 3 = hi/lo split of both operands (fp32-level accuracy), 1 = the leading TF32 parts only
int launch_gemm_tc(void* stream, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k, const float* a, int64_t lda,
                   const float* b, int64_t ldb, float* c, int64_t ldc, int32_t accumulate, int32_t epi, const float* aux,
                   int64_t ldaux, void* workspace, size_t workspace_bytes, int terms = 3, float* colsum_partial = nullptr,
                   const float* post_scale = nullptr);
// C = (A B^T) .* [mask > 0], out (+)= column sums of C, then (row_scale given) row i of C times row_scale[i]: the
// gradient of a hidden layer, its bias gradient and the scaled copy the next sparse product reads, in one pass
// over C when the tensor-core kernel takes the product (otherwise the product and the column-sum kernel).
// scratch: gemm_colsum_scratch(m, n) bytes.
int launch_gemm_mask_colsum(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k,
                            const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc,
                            const float* mask, int64_t ldmask, const float* row_scale, float* out, int32_t accumulate,
                            void* scratch, void* workspace, size_t workspace_bytes);
size_t gemm_colsum_scratch(int64_t m, int32_t n);
int64_t gemm_tc_colsum_rows(int64_t m);
size_t gemm_tc_workspace(int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k);
int launch_splitk_reduce(void* stream, int64_t m, int64_t n, int splits, const float* partial, int64_t ldp, float* c,
                         int64_t ldc,
                         int accumulate, int epi, const float* aux, int64_t ldaux);
// gather-rate probe (kernels_probe.cu): sms * 12 blocks of 8 warps; out = 128 floats per warp
int gather_probe_warps(int sms);
int launch_gather_probe(void* stream, const float* x, int64_t ldx, int64_t n_rows, int32_t window_rows, int32_t hit_every,
                        int32_t rounds, float* out, int sms);
int tc_status(int* out);  // error word of the tensor-core kernels (0 = no wait ran out)
int tc_clear();           // sets that word back to 0
int launch_softmax_ce(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                      const uint8_t* mask, int64_t n_train, float* loss_dev, float* grad, int64_t ldg, void* scratch);
size_t softmax_ce_scratch(int64_t n);
int launch_colsum(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                  void* scratch);
// the same sums, and on the way scaled[i, :] = rscale[i] * g[i, :] (scaled may be g)
int launch_colsum_scaled(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                         void* scratch, const float* rscale, float* scaled, int64_t lds);
size_t colsum_scratch(int64_t n, int32_t f);
int launch_adam(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m, float lr,
                float beta1, float beta2, float eps, int64_t t);
// pred[i] = argmax_j logits[i, j] (lowest j on ties); hits[b] = per-block count of masked rows with pred == y
int launch_argmax_hits(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                       const uint8_t* mask, int32_t* pred, int32_t* hits, int* n_blocks_out);
// device-resident step counter and bias corrections (state[0] = t, state[1..2] = 1 / (1 - beta^t))
int launch_adam_advance(void* stream, double* state, float beta1, float beta2);
int launch_adam_dev(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m, float lr,
                    float beta1, float beta2, float eps, const double* state);
// one partition's own Adam step from theta (not written): acc (+)= theta_p * inv_m; gsum cleared
int launch_adam_local_dev(void* stream, int64_t count, const float* theta, float* gsum, float* m, float* v, float* acc,
                          int first, float inv_m, float lr, float beta1, float beta2, float eps, const double* state);
int launch_normalize(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const int32_t* deg,
                     float* val);
int launch_inv_sqrt_degree(void* stream, int64_t n, const int32_t* deg, float* dinv);  // dinv[i] = 1 / sqrt(deg[i])
// dst[i, 0 .. f) = scale[i] * src[i, 0 .. f) (whole float4 chunks; leading dimensions multiples of 4; dst may be src)
int launch_scale_rows(void* stream, int64_t n, int32_t f, const float* scale, const float* src, int64_t lds, float* dst,
                      int64_t ldd);
// dst[i * ld + j] = src[i * f + j]: dense rows into padded rows
int launch_repitch(void* stream, int64_t n, int32_t f, const float* src, float* dst, int64_t ld);
int launch_mean(void* stream, const float* src, int count, float* dst);  // dst[0] = mean(src[0..count))

}  // namespace gcnsa
