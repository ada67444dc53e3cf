/*
 * gcnsa - full-batch GCN training on graph partitions augmented by subgraph
 * approximation, for one NVIDIA B200 (sm_100a).
 *
 * The method: a graph is split into M partitions; every partition p is extended
 * with a breadth-first random sample of at most nts = O N_p / (M - 1) vertices
 * from each other partition (Algorithm 1, Section 3.1); the edges among the
 * vertices of an extended partition are kept and all others dropped (Section
 * 4); a Kipf-Welling GCN, H^l = sigma(A_hat H^{l-1} W^l) (Section 4.1), is
 * trained on every extended partition and the results are averaged once per
 * epoch (Section 3.2; here the partition gradients are averaged in device
 * memory and one Adam step follows).
 *
 * Conventions
 *  - Every function returns GCNSA_OK (0) or a negative GCNSA_ERR_* code.  No
 *    function throws, aborts or prints.  gcnsa_last_error() gives a
 *    thread-local text for the most recent failure on the calling thread.
 *  - "host" / "device" is said for every pointer.  Host inputs stay the
 *    caller's and are not referenced after the call returns.  Everything the
 *    library allocates on the device goes through gcnsa_env.alloc / .free (or
 *    cudaMalloc / cudaFree when they are NULL) and is released by *_destroy.
 *  - All device work is enqueued on gcnsa_env.stream.  gcnsa_forward,
 *    gcnsa_backward, gcnsa_step and gcnsa_epoch are asynchronous; build, export
 *    and get synchronize the stream.
 *  - Dense matrices are row-major fp32.  Device matrices owned by the library
 *    use a leading dimension of GCNSA_LD(f) floats (f rounded up to a multiple
 *    of 16, so every row starts on a 64-byte boundary); the pad columns up to
 *    the next multiple of 4 hold zeros, the ones beyond are never read.
 *  - Sparse matrices are CSR with int32 row pointers and int32 column indices,
 *    columns ascending in each row.
 *  - Without a CUDA device of compute capability 10.x every call that needs
 *    the GPU fails with GCNSA_ERR_UNSUPPORTED_ARCH or GCNSA_ERR_CUDA; there is
 *    no CPU fallback.
 */
#ifndef GCNSA_H
#define GCNSA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GCNSA_OK 0
#define GCNSA_ERR_ARG (-1)              /* NULL / negative / inconsistent argument, unsorted row   */
#define GCNSA_ERR_NOT_SYMMETRIC (-2)    /* edge (u,v) without (v,u)                                */
#define GCNSA_ERR_SELF_LOOP_OR_DUP (-3) /* the input graph must be simple                          */
#define GCNSA_ERR_LABEL_RANGE (-4)      /* a label outside [0, c) or a partition id outside [0, m) */
#define GCNSA_ERR_OOM (-5)              /* host or device allocation failed                        */
#define GCNSA_ERR_ORDER (-6)            /* backward without forward, step with != M partitions...  */
#define GCNSA_ERR_CUDA (-7)             /* a CUDA call failed; text in gcnsa_last_error()          */
#define GCNSA_ERR_UNSUPPORTED_ARCH (-8) /* the current device is not sm_100                        */
#define GCNSA_ERR_TOO_LARGE (-9)        /* an extended partition exceeds int32 indexing            */

#define GCNSA_LD(f) ((((int64_t)(f)) + 15) / 16 * 16)
#define GCNSA_MAX_LAYERS 8

#define GCNSA_PART_RANGE 0 /* part[v] = floor(v M / N)                                     */
#define GCNSA_PART_HASH 1  /* rank by the 64-bit key, then the same rule on the rank       */
#define GCNSA_PART_USER 2  /* caller's array (how a METIS assignment is passed in)         */

#define GCNSA_BUILD_DEVICE 0 /* the master step runs in CUDA kernels (default)                  */
#define GCNSA_BUILD_HOST 1   /* the master step runs on the host cores, results are uploaded;  */
                             /* same results bit for bit                                       */

#define GCNSA_GEMM_FP32 0   /* fp32 FMA on the CUDA cores                                  */
#define GCNSA_GEMM_TF32X3 1 /* tcgen05 tensor cores, every operand split into two TF32    */
                            /* terms (three products): fp32-level accuracy; shapes the    */
                            /* tensor-core kernel cannot take run as GCNSA_GEMM_FP32      */
#define GCNSA_GEMM_TF32 2   /* the same kernel issuing one TF32 product per term: about   */
                            /* 3e-4 of the largest entry off, outside the 1e-4 bar the    */
                            /* training path is held to; kept to measure that             */

#define GCNSA_AGG_GRAD_AVG 0  /* partition gradients averaged in device memory, one Adam step    */
#define GCNSA_AGG_PARAM_AVG 1 /* Section 3.2 as written: every partition takes its own Adam    */
                              /* step from the aggregated parameters (own Adam state), and the */
                              /* resulting parameters are averaged                             */

typedef struct gcnsa_parts gcnsa_parts; /* all extended partitions, device resident         */
typedef struct gcnsa_model gcnsa_model; /* weights, Adam state, gradient sum, work buffers  */

/* Device memory and stream come from the caller (PyTorch in the Python binding). */
typedef struct {
  void* (*alloc)(size_t bytes, void* user); /* device pointer, 256-byte aligned, NULL on failure; may be NULL */
  void (*free)(void* dptr, void* user);     /* may be NULL iff alloc is NULL                                  */
  void* user;
  void* stream; /* cudaStream_t; NULL = the legacy default stream */
  int32_t device;
} gcnsa_env;

/* The whole graph G = (V, E), features X and labels (Section 2.1): HOST pointers. */
typedef struct {
  int64_t n, nnz;            /* vertices; directed non-zeros (both directions of each edge) */
  const int64_t* rowptr;     /* [n + 1]                                                     */
  const int32_t* col;        /* [nnz] ascending in each row; simple, symmetric, no loops    */
  int32_t f;                 /* feature width                                               */
  const float* x;            /* [n x f] row-major with leading dimension ldx >= f           */
  int64_t ldx;
  int32_t c;                 /* number of classes                                           */
  const int32_t* y;          /* [n] labels in [0, c)                                        */
  const uint8_t* train_mask; /* [n] 1 = training vertex                                     */
} gcnsa_graph;

typedef struct {
  int32_t m;                /* number of partitions M >= 1                                  */
  uint32_t overlap_ppm;     /* overlap threshold O of Algorithm 1 in parts per million      */
  uint64_t seed;            /* seed of the selection keys                                   */
  int32_t part_mode;        /* GCNSA_PART_*                                                 */
  const int32_t* user_part; /* HOST [n] when part_mode == GCNSA_PART_USER                   */
  int32_t loss_on_halo;     /* 1: sampled vertices that are training vertices carry loss    */
  int32_t builder;          /* GCNSA_BUILD_*: where gcnsa_build_partitions does its work    */
  int32_t order_window;     /* rows per window of the processing order (see                 */
                            /* gcnsa_part_schedule_host): 0 = the library decides (8192 for */
                            /* partitions of at least 131072 rows, whose gathered matrix    */
                            /* can exceed L2; one window otherwise), negative = one window  */
                            /* over all rows, otherwise at least 256.  Scheduling only: the */
                            /* results do not change                                        */
} gcnsa_part_opts;

typedef struct {
  int64_t n_owned, n_halo, n, nnz; /* rows owned, rows sampled in, n = sum, non-zeros of A + I */
  int64_t nts;                     /* vertices wanted from each other partition                */
  int64_t n_train;                 /* |T_p|: vertices carrying loss                            */
  int32_t max_depth;               /* deepest BFS level Algorithm 1 reached for this p         */
} gcnsa_part_info;

/* Caller-provided HOST buffers for gcnsa_parts_export_schedule; any may be NULL
 * (skipped).  These are the library's own scheduling structures: the order in
 * which the product kernels visit rows (hub rows first; then the other rows
 * window by window, a window being order_window consecutive rows, which bounds
 * the source rows that are live in L2 at any time; inside a window by
 * descending length class - lengths that agree in their five leading bits -
 * ties by row index) and the transposed CSR restricted to the columns that
 * carry loss. */
typedef struct {
  int32_t* order;     /* [n]        rows of A_hat in processing order                      */
  int32_t* t_order;   /* [n]        rows of the transposed CSR in processing order         */
  int32_t* m_order;   /* [n_train]  the rows that carry loss, in the order of `order`      */
  int32_t* tm_rowptr; /* [n + 1]    transposed CSR over the columns that carry loss        */
  int32_t* tm_col;    /* [tm_nnz]                                                          */
  int32_t* tm_order;  /* [n]        its rows in processing order                           */
  uint8_t* mask;      /* [n]        1 = the row carries loss                               */
  int32_t* y;         /* [n]        labels in partition order                              */
} gcnsa_part_schedule_host;

typedef struct {
  int64_t n_long, t_n_long, m_n_long, tm_n_long; /* hub rows at the head of each order       */
  int64_t m_nnz, tm_nnz;                         /* non-zeros in the loss rows / loss columns */
} gcnsa_part_schedule_info;

/* Caller-provided HOST buffers for gcnsa_parts_export; any may be NULL (skipped). */
typedef struct {
  int32_t* rowptr;   /* [n + 1]  */
  int32_t* col;      /* [nnz]    */
  float* val;        /* [nnz]    */
  int32_t* t_rowptr; /* [n + 1]  transposed CSR */
  int32_t* t_col;    /* [nnz]    */
  float* t_val;      /* [nnz]    */
  int64_t* members;  /* [n] local -> global id: owned ascending, then sampled ascending */
  int32_t* depth;    /* [m] BFS levels used per other partition (0 for p itself)        */
} gcnsa_part_host;

typedef struct {
  int32_t n_layers;                   /* L in [1, GCNSA_MAX_LAYERS]                           */
  int32_t dims[GCNSA_MAX_LAYERS + 1]; /* dims[0] = f, dims[L] = c                             */
  int32_t use_bias;
  float lr, beta1, beta2, eps;        /* Adam; the paper fixes lr = 0.02 (Section 4.1)        */
  int32_t gemm_mode;                  /* GCNSA_GEMM_*                                         */
  int32_t agg_mode;                   /* GCNSA_AGG_*                                          */
  int32_t loss_rows_only;             /* 1: gcnsa_forward computes the last layer only on the  */
                                      /* rows that carry loss (training reads no others; the   */
                                      /* other rows of GCNSA_GET_ACT(L) are then undefined);   */
                                      /* 0: every row.  gcnsa_evaluate always computes all.    */
  int32_t epoch_graph;                /* 1: gcnsa_epoch records its kernel sequence into a     */
                                      /* CUDA graph on first use and replays it afterwards     */
                                      /* (needs a stream other than the legacy default stream; */
                                      /* falls back to plain launches otherwise or while       */
                                      /* gcnsa_model_profile is on).  Results are identical.   */
  int32_t factored_norm;              /* 1: layers that multiply by W first compute            */
                                      /* A_hat T as diag(d^-1/2) (A + I) (diag(d^-1/2) T): the */
                                      /* rows of T are scaled in one pass, the sparse product  */
                                      /* reads no values (one load less per non-zero) and      */
                                      /* scales its result rows.  Same sums up to fp32         */
                                      /* rounding (1e-7 relative).  0: stored values are read. */
  int32_t cache_ax;                   /* 1: the first layer runs as (A_hat X) W and A_hat X of  */
                                      /* every partition is kept in device memory (n_p x LD(f)  */
                                      /* floats each) for as long as the feature rows are not   */
                                      /* rewritten: A_hat and X are constants of the training,   */
                                      /* so after the first epoch layer 1 needs no sparse        */
                                      /* product in either direction.  Same arithmetic as the    */
                                      /* paper's H^1 = sigma(A_hat X W^1); an algebraic shortcut  */
                                      /* that skips the per-epoch product, hence off by default. */
} gcnsa_model_opts;

const char* gcnsa_strerror(int code);
const char* gcnsa_last_error(void);
/* Number of kernels this library has launched since it was loaded (all threads). */
int64_t gcnsa_launch_count(void);
/* How the dense products (the feature transform H W of Section 4.1 and its
 * gradient products) asked for in GCNSA_GEMM_TF32X3 mode were run since the
 * library was loaded: *tensor_core counts those the tcgen05 kernel took,
 * *fp32_fallback those that ran on the fp32 FMA kernel instead because the
 * tensor-core path could not take them (an operand base or pitch that is not
 * 16-byte aligned, too little workspace, no tensor-map encoder in the driver).
 * Products recorded into a CUDA graph are counted once, when recorded.
 * Products asked for in GCNSA_GEMM_FP32 mode count in neither.  HOST pointers. */
int gcnsa_gemm_path_counts(int64_t* tensor_core, int64_t* fp32_fallback);
/* Fills *opts with the configuration the published throughput figures of this
 * library belong to: two layers (set n_layers and dims yourself), bias on, Adam
 * with lr 0.02 (Section 4.1), beta1 0.9, beta2 0.999, eps 1e-8,
 * GCNSA_GEMM_TF32X3, GCNSA_AGG_GRAD_AVG, loss_rows_only = 1, epoch_graph = 1,
 * factored_norm = 1, cache_ax = 0.  A zeroed gcnsa_model_opts instead selects
 * the plainest path (fp32 FMA products, stored values read, every row of the
 * last layer computed, plain launches), which the parity tests also cover. */
void gcnsa_model_opts_default(gcnsa_model_opts* opts);

/*
 * Master initialisation (Section 3.2): partition assignment (Section 4, METIS
 * replaced by a seeded stand-in or a caller-provided assignment), Algorithm 1
 * for every ordered pair (p, op) read as breadth-first levels with "random"
 * realised as the nts smallest unique 64-bit keys, the graph induced on every
 * extended partition plus self-loops (Section 3.1 step 2, Section 4), its
 * D^-1/2 (A + I) D^-1/2 weights with degrees counted inside the extended
 * partition (Section 4.1 footnote), the transposed CSR, and the feature /
 * label / mask rows gathered into partition order.  All results are resident
 * in device memory when the call returns.
 *
 * With GCNSA_BUILD_DEVICE the graph, features, labels and mask are uploaded
 * once and every step above runs in CUDA kernels: checks of the input graph,
 * the assignment, the breadth-first levels of Algorithm 1 for all other
 * partitions at once, the key selection (a radix select over the 64-bit keys),
 * the induced rows, the transpose (a stable radix sort by column) and the row
 * orders.  The host only reads back sizes to allocate the results.  Needs
 * about 8 (n + nnz) + 4 n f bytes of device memory for the inputs plus 24 bytes
 * per non-zero of the largest partition as scratch, released before returning.
 * GCNSA_BUILD_HOST computes the structure on the host cores instead.
 */
int gcnsa_build_partitions(const gcnsa_env* env, const gcnsa_graph* g, const gcnsa_part_opts* opts,
                           gcnsa_parts** out);
/*
 * The same master step without a device: partition assignment, Algorithm 1 and
 * the structure of every extended partition, computed and kept in HOST memory.
 * Lets a caller size device memory (rows and non-zeros per partition) before
 * building, and inspect what Algorithm 1 selected.  Needs no GPU.
 * gcnsa_plan_export fills rowptr, col, t_rowptr, t_col, members and depth; val
 * and t_val are computed on the device only and are left untouched.
 */
typedef struct gcnsa_plan gcnsa_plan;
int gcnsa_plan_create(const gcnsa_graph* g, const gcnsa_part_opts* opts, gcnsa_plan** out);
int gcnsa_plan_info(const gcnsa_plan* plan, int32_t p, gcnsa_part_info* out);
int gcnsa_plan_assignment(const gcnsa_plan* plan, int32_t* part_host /* [n] */);
int gcnsa_plan_export(const gcnsa_plan* plan, int32_t p, const gcnsa_part_host* dst);
/* The scheduling structures as the host cores compute them (mask and y of dst are
 * not filled: labels are gathered on the device only). */
int gcnsa_plan_export_schedule(const gcnsa_plan* plan, int32_t p, gcnsa_part_schedule_info* info,
                               const gcnsa_part_schedule_host* dst);
int gcnsa_plan_destroy(gcnsa_plan* plan);

int gcnsa_parts_count(const gcnsa_parts* parts);
int gcnsa_parts_info(const gcnsa_parts* parts, int32_t p, gcnsa_part_info* out);
int gcnsa_parts_assignment(const gcnsa_parts* parts, int32_t* part_host /* [n] */);
int gcnsa_parts_export(const gcnsa_parts* parts, int32_t p, const gcnsa_part_host* dst);
/* The scheduling structures of partition p (sizes in *info, which may be asked for
 * alone with dst == NULL).  Synchronizes the stream. */
int gcnsa_parts_export_schedule(const gcnsa_parts* parts, int32_t p, gcnsa_part_schedule_info* info,
                                const gcnsa_part_schedule_host* dst);
/* Copies partition p's feature rows ([n_p x f], leading dimension f) into HOST memory. */
int gcnsa_parts_get_features(const gcnsa_parts* parts, int32_t p, float* x_host);
/* Replace the device copy of partition p's feature rows from HOST memory
 * ([n_p x f] row-major, leading dimension f, partition order); asynchronous on
 * the stream, so x_host must stay valid until the stream reaches the copy. */
int gcnsa_parts_set_features(gcnsa_parts* parts, int32_t p, const float* x_host);
int gcnsa_parts_destroy(gcnsa_parts* parts);

/* w0[l]: HOST [dims[l] x dims[l+1]] row-major; b0[l]: HOST [dims[l+1]] (NULL = zeros). */
int gcnsa_model_create(const gcnsa_env* env, const gcnsa_parts* parts, const gcnsa_model_opts* opts,
                       const float* const* w0, const float* const* b0, gcnsa_model** out);

/*
 * Forward pass on extended partition p (Section 4.1): for every layer
 * Z = A_hat H W + b, ReLU between layers, masked softmax cross-entropy on the
 * last layer.  Each layer multiplies in the cheaper order (H W first when the
 * layer narrows, A_hat H first when it widens).  loss_dev: nullable DEVICE
 * float that receives the mean loss over T_p.
 */
int gcnsa_forward(gcnsa_model* model, const gcnsa_parts* parts, int32_t p, float* loss_dev);
/* Backward pass for the partition of the latest gcnsa_forward; adds dW, db into
 * the gradient sum.  The transposed product runs over the prebuilt transposed
 * CSR: no atomics, results are run-to-run identical. */
int gcnsa_backward(gcnsa_model* model, const gcnsa_parts* parts, int32_t p);
/* Epoch-end aggregation (Section 3.2).  GCNSA_AGG_GRAD_AVG: g = sum / M, one
 * Adam step with bias correction, gradient sum cleared.  GCNSA_AGG_PARAM_AVG:
 * every gcnsa_backward has already taken partition p's own Adam step from the
 * aggregated parameters and added the result / M to an accumulator; the step
 * makes that mean the new parameters.  Requires exactly M backward passes. */
int gcnsa_step(gcnsa_model* model);
/* forward + backward for p = 0..M-1, then step.  loss_dev: nullable DEVICE
 * float, mean of the M partition losses. */
int gcnsa_epoch(gcnsa_model* model, const gcnsa_parts* parts, float* loss_dev);
/* The same epoch driven from HOST buffers: x_host[p] (partition order, as for
 * gcnsa_parts_set_features; pinned memory lets the copies overlap compute) is
 * uploaded before partition p is used and the epoch loss is copied to
 * *loss_host; returns after the stream has drained. */
int gcnsa_epoch_host(gcnsa_model* model, gcnsa_parts* parts, const float* const* x_host, float* loss_host);

/* Per-kernel timing of forward / backward / step with CUDA events on the
 * model's stream.  Classes: 0 = SpMM, 1 = GEMM, 2 = everything else.  alg_bytes
 * is the compulsory memory traffic of the launches (SpMM: row pointers, column
 * indices, values, one read of the source rows, one write of the result);
 * l1_bytes is what the SMs must pull through their L1 data path (SpMM: the same
 * with one gather of a source row per stored entry, 4 f nnz, in place of the one
 * read of the source rows; equal to alg_bytes for the other classes);
 * alg_bytes_val is alg_bytes with 8 bytes per stored entry (index and value)
 * whether or not the kernel in use reads values; flops counts multiply-adds
 * as 2. */
typedef struct {
  double ms[3];
  int64_t launches[3];
  double alg_bytes[3];
  double flops[3];
  double l1_bytes[3];
  double alg_bytes_val[3];
} gcnsa_profile;
int gcnsa_model_profile(gcnsa_model* model, int32_t enable);
/* Synchronizes the stream, sums what was recorded since the last read, clears. */
int gcnsa_model_profile_read(gcnsa_model* model, gcnsa_profile* out);

/*
 * Evaluation (Section 2.2: micro-F1, which for one label per vertex is the
 * accuracy).  Runs the forward pass of the current parameters on partition p of
 * `parts` (typically partitions built with m = 1 and no overlap: the complete
 * graph), takes the row-wise argmax of the last layer (ties to the lowest
 * class) and counts the vertices of `mask_host` (HOST [n_p] in partition order;
 * NULL = all) whose prediction equals their label.  pred_host (nullable, HOST
 * [n_p]) receives the predictions.  micro-F1 = *correct / *total.
 * Synchronizes the stream; the model must have been created for partitions at
 * least as large.
 */
int gcnsa_evaluate(gcnsa_model* model, const gcnsa_parts* parts, int32_t p, const uint8_t* mask_host,
                   int64_t* correct_host, int64_t* total_host, int32_t* pred_host);
/* Copies weights and biases (not the optimizer state) from a model with the same dims. */
int gcnsa_model_copy_params(gcnsa_model* dst, const gcnsa_model* src);

/* ---- GraphSAGE with the mean aggregator (Section 4.1, "Investigated GCNs") ----
 *
 * The paper's second model: a fixed number of neighbours is sampled per vertex,
 * their features are averaged element-wise, 2 layers, mini-batches (256 in the
 * paper), Adam; every worker trains its own copy of the parameters on its
 * extended partition for an epoch and the copies are averaged (Section 3.2).
 * Where the paper is silent this library takes:
 *  - layer  h_v = sigma(h_v W_self + mean_{u in S(v)} h_u W_neigh + b), ReLU after
 *    the first layer, softmax cross-entropy on the second; no normalisation of
 *    the embeddings;
 *  - S(v): uniform without replacement among the neighbours of v inside its
 *    extended partition (v excluded), all of them when there are at most
 *    fanout; realised as the fanout smallest 64-bit selection keys, a function
 *    of (seed, partition, epoch, layer, v) only; no neighbours: mean = 0;
 *  - batches: the loss-carrying vertices of the partition in ascending order of
 *    a second key (seed, partition, epoch), cut into groups of `batch`;
 *  - one Adam step per batch on the worker's copy, Adam state per worker kept
 *    across epochs; epoch loss = mean over partitions of the batch losses
 *    weighted by batch size.
 */
typedef struct {
  int32_t dims[3];   /* f, hidden width, c                                               */
  int32_t fanout[2]; /* neighbours sampled by the hidden layer, by the output layer       */
  int32_t batch;     /* vertices per mini-batch                                           */
  float lr, beta1, beta2, eps;
  uint64_t seed;     /* seed of the sampling and batching keys                            */
  int32_t gemm_mode; /* GCNSA_GEMM_*                                                      */
  int32_t batch_graph; /* 1: gcnsa_sage_epoch records the kernel sequence of a worker's full-size
                        * batch once (CUDA graph) and replays it, the batch index and the epoch
                        * living in device memory; the ragged last batch and gcnsa_sage_batch
                        * use plain launches.  Same results bit for bit.  Needs a stream other
                        * than the legacy default stream; otherwise plain launches. */
} gcnsa_sage_opts;
typedef struct gcnsa_sage gcnsa_sage;

/* w_self0[l], w_neigh0[l]: HOST [din x dout] row-major for l = 0 (f x hidden) and
 * l = 1 (hidden x c); b0 (nullable, entries nullable): HOST [dout], zeros otherwise. */
int gcnsa_sage_create(const gcnsa_env* env, const gcnsa_parts* parts, const gcnsa_sage_opts* opts,
                      const float* const* w_self0, const float* const* w_neigh0, const float* const* b0,
                      gcnsa_sage** out);
/* One epoch (Section 3.2): for every partition the worker's copy is set to the
 * aggregated parameters and takes one Adam step per batch; afterwards the
 * aggregated parameters become the mean of the copies.  loss_dev: nullable
 * DEVICE float, the epoch loss.  Asynchronous on the stream. */
int gcnsa_sage_epoch(gcnsa_sage* model, const gcnsa_parts* parts, float* loss_dev);
int gcnsa_sage_get_epoch(const gcnsa_sage* model, int64_t* epoch_out); /* epochs run so far = index of the next */
/* Timing of the batches with CUDA events on the model's stream, as
 * gcnsa_model_profile does for the Kipf-Welling path.  Classes: 0 = the gathers
 * that assemble the [self | mean] rows (alg_bytes: every source row read - the
 * vertex's own and each sampled neighbour's, counted on the device - plus the
 * rows written), 1 = dense products (flops), 2 = everything else (sampling,
 * loss, bias gradients, Adam). */
int gcnsa_sage_profile(gcnsa_sage* model, int32_t enable);
int gcnsa_sage_profile_read(gcnsa_sage* model, gcnsa_profile* out);
/* Number of batches of partition p. */
int gcnsa_sage_batches(const gcnsa_sage* model, const gcnsa_parts* parts, int32_t p, int64_t* count_out);
/* Batch b of partition p as epoch `epoch` would run it, on the working copy of
 * the parameters as it stands: forward, loss, backward; apply != 0 also takes
 * worker p's Adam step.  loss_dev: nullable DEVICE float, the batch loss.  For
 * tests and step-by-step use; gcnsa_sage_epoch is the training call. */
int gcnsa_sage_batch(gcnsa_sage* model, const gcnsa_parts* parts, int32_t p, int64_t epoch, int64_t b, int32_t apply,
                     float* loss_dev);
/* The latest batch: nb vertices and rows1 = nb (1 + fanout[1]) rows of the hidden
 * layer (row i < nb is batch vertex i, row nb + i fanout[1] + s its s-th sampled
 * neighbour of the output layer, or no vertex).  Caller-provided HOST buffers,
 * any may be NULL.  Synchronizes the stream. */
typedef struct {
  int32_t* vertices; /* [rows1]             local vertex id per row, -1 = none               */
  int32_t* count2;   /* [nb]                neighbours the output layer sampled per vertex   */
  int32_t* samples1; /* [rows1 x fanout[0]] neighbours the hidden layer sampled, -1 padded   */
  int32_t* count1;   /* [rows1]                                                              */
  float* hidden;     /* [rows1 x hidden]    embeddings after the first layer                 */
  float* logits;     /* [nb x c]                                                             */
  float* dlogits;    /* [nb x c]            gradient of the batch loss w.r.t. the logits     */
  float* loss;       /* [1]                 batch loss                                       */
} gcnsa_sage_batch_host;
int gcnsa_sage_batch_shape(const gcnsa_sage* model, int64_t* nb_out, int64_t* rows1_out);
int gcnsa_sage_batch_export(const gcnsa_sage* model, const gcnsa_sage_batch_host* dst);
#define GCNSA_SAGE_W_SELF 0       /* aggregated parameters, layer l: [din x dout]              */
#define GCNSA_SAGE_W_NEIGH 1
#define GCNSA_SAGE_B 2            /* [dout]                                                    */
#define GCNSA_SAGE_WORK_W_SELF 3  /* the working copy (the worker that ran last)               */
#define GCNSA_SAGE_WORK_W_NEIGH 4
#define GCNSA_SAGE_WORK_B 5
#define GCNSA_SAGE_GRAD_W_SELF 6  /* gradient of the latest batch (zero after an Adam step)    */
#define GCNSA_SAGE_GRAD_W_NEIGH 7
#define GCNSA_SAGE_GRAD_B 8
/* Copy one tensor into HOST memory (dense, no padding); bytes must match. */
int gcnsa_sage_get(const gcnsa_sage* model, int32_t what, int32_t layer, void* host_dst, size_t bytes);
int gcnsa_sage_destroy(gcnsa_sage* model);

#define GCNSA_GET_W 0        /* layer l: [dims[l] x dims[l+1]]                              */
#define GCNSA_GET_B 1        /* layer l: [dims[l+1]]                                        */
#define GCNSA_GET_GRAD_W 2   /* gradient sum, same shapes                                   */
#define GCNSA_GET_GRAD_B 3
#define GCNSA_GET_ADAM_M_W 4
#define GCNSA_GET_ADAM_M_B 5
#define GCNSA_GET_ADAM_V_W 6
#define GCNSA_GET_ADAM_V_B 7
#define GCNSA_GET_ACT 8      /* H^l of the latest forward, l in [1, L]: [n_p x dims[l]]     */
#define GCNSA_GET_DLOGITS 9  /* gradient of the loss w.r.t. the logits: [n_p x c]           */
/* Copy one tensor into HOST memory (dense, no padding); bytes must match. */
int gcnsa_model_get(const gcnsa_model* model, int32_t what, int32_t layer, void* host_dst, size_t bytes);
int gcnsa_model_set(gcnsa_model* model, int32_t what, int32_t layer, const void* host_src, size_t bytes);
/* With GCNSA_AGG_PARAM_AVG every partition has its own Adam moments: choose whose
 * moments GCNSA_GET_ADAM_* / gcnsa_model_set address (partition 0 after create). */
int gcnsa_model_select_partition(gcnsa_model* model, int32_t p);
int gcnsa_model_get_t(const gcnsa_model* model, int64_t* t_out);
int gcnsa_model_set_t(gcnsa_model* model, int64_t t);
int gcnsa_model_destroy(gcnsa_model* model);

/* ---- single operations on caller-owned DEVICE buffers (tests, sweeps) ---- */

#define GCNSA_EPI_NONE 0
#define GCNSA_EPI_BIAS 1      /* + bias[j]                                                   */
#define GCNSA_EPI_BIAS_RELU 2 /* max(. + bias[j], 0); bias may be NULL                       */
#define GCNSA_EPI_MASK 3      /* multiplied by [mask[i, j] > 0] (ReLU derivative)            */
#define GCNSA_EPI_ROWSCALE 4  /* row i multiplied by aux[i] (gcnsa_op_gemm only): the d^-1/2 */
                              /* of the factored normalization applied by the producer       */

/* Y = epi(A X): the normalized-adjacency product of Section 4.1 (and, given the
 * transposed CSR, of its backward pass).  rowptr/col/val DEVICE CSR with n_rows
 * rows; order: nullable DEVICE permutation of the rows giving the processing
 * order (longest rows first balances a power-law graph); n_long: the first
 * n_long rows of order get a whole thread block each instead of a warp (hub
 * rows; 0 = none); x, y: DEVICE [. x f] with leading dimensions ldx, ldy (multiples of 4,
 * 16-byte aligned bases; columns f..ld of x must be zero); aux: bias [f] or
 * mask [n_rows x ldaux] per epi.  x and y must not overlap. */
int gcnsa_op_spmm(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const float* val,
                  const int32_t* order, int64_t n_long, const float* x, int64_t ldx, int32_t f, int32_t epi, const float* aux,
                  int64_t ldaux, float* y, int64_t ldy);

/* Y = epi(diag(row_scale) B X) where B is the 0/1 pattern of the CSR: no values
 * are read, every stored entry counts as 1.  Because A_hat = D^-1/2 (A + I) D^-1/2
 * (Section 4.1 footnote), A_hat X = diag(d^-1/2) B (diag(d^-1/2) X): with the
 * source rows scaled beforehand and row_scale = d^-1/2 this is the same product
 * as gcnsa_op_spmm with one load less per non-zero.  row_scale: nullable DEVICE
 * [n_rows]; everything else as for gcnsa_op_spmm. */
int gcnsa_op_spmm_pattern(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col,
                          const float* row_scale, const int32_t* order, int64_t n_long, const float* x, int64_t ldx,
                          int32_t f, int32_t epi, const float* aux, int64_t ldaux, float* y, int64_t ldy);

/* C = epi(op(A) op(B)) (+ C when accumulate): the dense feature transform H W
 * and the gradient products H^T dT, dT W^T.  op(A) is m x k, op(B) is k x n;
 * ta / tb = 1 means the stored matrix is the transpose.  All DEVICE, row-major.
 * workspace: DEVICE scratch, 256-byte aligned, of at least
 * gcnsa_op_gemm_workspace() bytes (may be NULL when that is 0; with less, the
 * product runs unsplit on the fp32 FMA kernel). */
int gcnsa_op_gemm(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k,
                  const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc,
                  int32_t accumulate, int32_t epi, const float* aux, int64_t ldaux, void* workspace,
                  size_t workspace_bytes);
size_t gcnsa_op_gemm_workspace(int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k);

/* The gradient of a hidden layer in one call (backward pass of the layer of
 * Section 4.1): C = (op(A) op(B)) .* [mask > 0] (the ReLU derivative),
 * out[j] (+)= sum_i C[i, j] (the bias gradient of the layer below), and, when
 * row_scale is given, row i of C is then multiplied by row_scale[i] (the d^-1/2
 * of the factored normalization that the next sparse product expects on its
 * source rows; the sums are those of the unscaled C).  On the tensor-core
 * kernel the sums and the scaling happen in the epilogue of the product; a
 * product that kernel cannot take runs as gcnsa_op_gemm followed by
 * gcnsa_op_colsum_scaled, with the same results up to rounding order.
 * mask: DEVICE [m x ldmask]; row_scale: nullable DEVICE [m]; out: DEVICE [n];
 * scratch: DEVICE, 256-byte aligned, gcnsa_op_gemm_mask_colsum_scratch(m, n)
 * bytes; workspace as for gcnsa_op_gemm.  Sums are added in a fixed order. */
int gcnsa_op_gemm_mask_colsum(void* stream, int32_t mode, int32_t ta, int32_t tb, int64_t m, int64_t n, int64_t k,
                              const float* a, int64_t lda, const float* b, int64_t ldb, float* c, int64_t ldc,
                              const float* mask, int64_t ldmask, const float* row_scale, float* out,
                              int32_t accumulate, void* scratch, size_t scratch_bytes, void* workspace,
                              size_t workspace_bytes);
size_t gcnsa_op_gemm_mask_colsum_scratch(int64_t m, int32_t n);
/* A measuring stick for gcnsa_op_spmm / gcnsa_op_spmm_pattern, not a step of
 * the method (the paper has no counterpart): the rate at which the SMs gather
 * 512-byte rows (the first 128 floats of a row of x) when the indices cost
 * nothing.  gcnsa_op_gather_probe_warps(&w) warps (12 blocks of 8 per SM) each
 * add up `rounds` x 16 rows; row k of a round is drawn from the warp's own
 * generator (s <- s * 1664525 + 1013904223 mod 2^32, s <- s ^ (s >> 15),
 * starting from 0x9E3779B9 * (warp + 1) mod 2^32; the row is floor(s * range /
 * 2^32)): from the block's window [base, base + window_rows), base = (block *
 * 977) mod (n_rows - window_rows + 1), when hit_every > 0 and k mod hit_every
 * = 0, otherwise from all n_rows rows.  hit_every = 0 measures the L2 -> L1
 * path without reuse, 1 the L1 data path alone, 4 a quarter of hits.  out:
 * DEVICE [warps x 128], the lane-wise sums (so that a test can check the
 * gathers).  x: DEVICE, 16-byte aligned, ldx >= 128 and a multiple of 4,
 * 1 <= window_rows <= n_rows < 2^31.  Timing is the caller's (events). */
int gcnsa_op_gather_probe(void* stream, const float* x, int64_t ldx, int64_t n_rows, int32_t window_rows,
                          int32_t hit_every, int32_t rounds, float* out, size_t out_bytes);
int gcnsa_op_gather_probe_warps(int32_t* warps_out);

/* The tensor-core kernels bound every wait (tens of milliseconds); a wait that
 * runs out stores a non-zero code in a device word instead of hanging.  The
 * word is sticky: while it is set, every tensor-core launch returns at once
 * without computing, so results after a non-zero status are undefined until
 * gcnsa_tc_clear.  gcnsa_tc_status synchronizes the device and copies the word
 * to *status_host (0 = healthy); gcnsa_tc_clear synchronizes and resets it. */
int gcnsa_tc_status(int32_t* status_host);
int gcnsa_tc_clear(void);
/* The checking build of the library (compiled with -DGCNSA_DEBUG into
 * libgcnsa_debug.so; the stand-in for a memory checker): the sparse product of
 * Section 4.1 checks every row of the processing order, every row range and
 * every gathered column index against the sizes of the extended partition, and
 * the kernels of gcnsa_build_partitions that scatter by computed positions
 * (induced rows of Section 3.1, the radix sort behind the transpose, the
 * transposed CSR over the loss columns) check every write position.  A failed
 * check records what it saw and skips the access; nothing traps.
 * *enabled_host = 1 in the checking build, 0 otherwise (then the rest is 0).
 * *code_host = 0 when every check passed, else 1 = processing-order entry,
 * 2 = row range, 3 = column index, 4 = induced-row write, 5 = sort scatter,
 * 6 = loss-column write; *value_host = the offending value.  Synchronizes the
 * device and clears the record.  HOST pointers. */
int gcnsa_debug_status(int32_t* enabled_host, int32_t* code_host, int64_t* value_host);

/* Masked softmax cross-entropy over n rows of c logits: *loss_dev = (1/n_train)
 * sum over masked rows of (logsumexp(z_i) - z_i[y_i]); grad = (softmax - onehot)
 * mask / n_train (zero rows elsewhere, pad columns zero).  n_train = 0 gives
 * loss 0 and a zero gradient.  scratch: DEVICE, gcnsa_op_softmax_ce_scratch(n)
 * bytes. */
int gcnsa_op_softmax_ce(void* stream, int64_t n, int32_t c, const float* logits, int64_t ld, const int32_t* y,
                        const uint8_t* mask, int64_t n_train, float* loss_dev, float* grad, int64_t ldg,
                        void* scratch, size_t scratch_bytes);
size_t gcnsa_op_softmax_ce_scratch(int64_t n);

/* out[j] (+)= sum_i g[i, j]: the bias gradient.  scratch: gcnsa_op_colsum_scratch(n, f) bytes. */
int gcnsa_op_colsum(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out, int32_t accumulate,
                    void* scratch, size_t scratch_bytes);
size_t gcnsa_op_colsum_scratch(int64_t n, int32_t f);
/* The same column sums, and in the same pass scaled[i, :] = row_scale[i] * g[i, :]
 * over whole float4 chunks (the d^-1/2 G the factored transposed product reads;
 * the bias gradient needs every element of G anyway).  g, scaled: 16-byte
 * aligned, leading dimensions multiples of 4 and at least f rounded up to 4;
 * scaled may be g (in place). */
int gcnsa_op_colsum_scaled(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out,
                           int32_t accumulate, void* scratch, size_t scratch_bytes, const float* row_scale,
                           float* scaled, int64_t lds);

/*
 * The same column sums for callers that must not allocate device memory:
 * code running while a CUDA graph is being captured elsewhere in the process,
 * inside another framework's memory pool whose allocator it may not re-enter,
 * or under a fixed memory budget where cudaMalloc may fail or stall the device.
 * (The paper has no counterpart; this is a convenience of the library.)
 * The scratch is a device array built into the library, 592 block slots x
 * GCNSA_COLSUM_STATIC_MAX_F floats (2.3 MiB; a call uses at most 296 of the
 * slots), present on every GPU that loads
 * the library until the process exits.  The call allocates and frees nothing.
 *  - f > GCNSA_COLSUM_STATIC_MAX_F returns GCNSA_ERR_TOO_LARGE: use
 *    gcnsa_op_colsum with your own scratch instead.
 *  - The first call on a device looks up the array's device address (no
 *    allocation); make that first call with the device current and before any
 *    stream capture begins.
 *  - All calls on a device share the one array, and it keeps the previous
 *    call's partial sums.  Each call overwrites every partial it later reads, so
 *    nothing has to be cleared; but two calls that can run on the GPU at the
 *    same time (different streams, no ordering between them) race on it.  Keep
 *    calls on one stream or order them with events.
 * Results equal gcnsa_op_colsum bit for bit (same kernels, same order).
 */
#define GCNSA_COLSUM_STATIC_MAX_F 1024
int gcnsa_op_colsum_static(void* stream, int64_t n, int32_t f, const float* g, int64_t ldg, float* out,
                           int32_t accumulate);

/* g = gsum * inv_m; Adam step number t (>= 1) on theta with moments m, v; gsum
 * cleared.  All DEVICE [count]. */
int gcnsa_op_adam(void* stream, int64_t count, float* theta, float* gsum, float* m, float* v, float inv_m,
                  float lr, float beta1, float beta2, float eps, int64_t t);

/* val[e] = 1 / sqrt(deg[i] deg[col[e]]) for e in row i: D^-1/2 (A+I) D^-1/2. */
int gcnsa_op_normalize(void* stream, int64_t n_rows, const int32_t* rowptr, const int32_t* col, const int32_t* deg,
                       float* val);

#ifdef __cplusplus
}
#endif
#endif /* GCNSA_H */
