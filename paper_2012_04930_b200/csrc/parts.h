// The device-resident partitions object and the allocator / stream wrapper,
// shared by the C-ABI translation unit and the device-side partition builder.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "internal.h"

namespace gcnsa {

struct Env {
  gcnsa_env e{};
  cudaStream_t stream() const { return (cudaStream_t)e.stream; }
  void* alloc(size_t bytes) const {
    if (bytes == 0) bytes = 256;
    if (e.alloc) return e.alloc(bytes, e.user);
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
  }
  void release(void* p) const {
    if (!p) return;
    if (e.alloc) e.free(p, e.user);
    else cudaFree(p);
  }
};

struct DevPart {
  gcnsa_part_info info{};
  int32_t *rowptr = nullptr, *col = nullptr, *t_rowptr = nullptr, *t_col = nullptr, *order = nullptr, *t_order = nullptr;
  float *val = nullptr, *t_val = nullptr, *x = nullptr;
  float* dinv = nullptr;  // d_i^-1/2 with d the row lengths of A + I (A_hat = diag(dinv) (A + I) diag(dinv))
  int32_t* m_order = nullptr;  // rows that carry loss, longest first
  int64_t m_n_long = 0, m_nnz = 0;
  int32_t *tm_rowptr = nullptr, *tm_col = nullptr, *tm_order = nullptr;  // transposed CSR over loss-carrying columns
  float* tm_val = nullptr;
  int64_t tm_nnz = 0, tm_n_long = 0;
  int32_t* y = nullptr;
  uint8_t* mask = nullptr;
  std::vector<int64_t> members;
  std::vector<int32_t> depth;
  int64_t n_long = 0, t_n_long = 0;
};

}  // namespace gcnsa

struct gcnsa_parts {
  gcnsa::Env env;
  int32_t m = 0, f = 0, c = 0;
  int64_t n = 0, ldx = 0, n_max = 0;
  int32_t builder = 0;  // GCNSA_BUILD_* that produced the object
  std::vector<int32_t> part;
  std::vector<gcnsa::DevPart> parts;
  std::vector<void*> owned;  // every device allocation, for destroy
  void* dalloc(size_t bytes) {
    void* p = env.alloc(bytes);
    if (p) owned.push_back(p);
    return p;
  }
  std::vector<int64_t> x_version;  // bumped whenever a partition's feature rows are rewritten
  uint64_t uid = 0;                // distinguishes partition objects that reuse an address
  // upload pipeline of gcnsa_epoch_host (created on first use)
  cudaStream_t copy_stream = nullptr;
  std::vector<cudaEvent_t> ready, consumed;
  float* staging[2] = {nullptr, nullptr};
};

namespace gcnsa {

// The master step on the device: assignment, Algorithm 1, induced CSR, transposed
// CSR, processing orders, feature / label / mask rows and A_hat values.  Fills
// P->part and P->parts (P->env, m, f, c, n, ldx set by the caller).  The graph
// arrays of g are HOST pointers; argument checks that need no device are done
// by the caller.
int build_device(gcnsa_parts* P, const gcnsa_graph* g, const gcnsa_part_opts* o);
// Argument checks of gcnsa_build_partitions that need neither the graph's contents nor a device.
int check_build_args(const gcnsa_graph* g, const gcnsa_part_opts* o);
// Host check that the CSR is a simple symmetric graph with ascending rows and labels in range.
int validate_graph_host(const gcnsa_graph* g);

}  // namespace gcnsa
