// Bounds checks of the index-driven kernels, compiled in with -DGCNSA_DEBUG (a
// library of its own, libgcnsa_debug.so).  A check that fails records a code
// and the offending value in a device word with one atomicCAS (the first
// failure wins) and the kernel skips that access: nothing traps, the context
// stays usable, the host reads the word with gcnsa_debug_status.  Without the
// macro every check is compiled out.
#pragma once
#include <cstdint>

namespace gcnsa {

// what was out of range (top byte of the word; the low 56 bits hold the value)
constexpr int kDbgOrderEntry = 1;    // a row of the processing order outside [0, rows of the matrix)
constexpr int kDbgRowRange = 2;      // rowptr[r] > rowptr[r + 1], negative, or beyond the stored entries
constexpr int kDbgColumn = 3;        // a column index outside [0, source rows)
constexpr int kDbgInducedWrite = 4;  // induced rows: a write position outside the row
constexpr int kDbgSortWrite = 5;     // radix sort: a scatter position outside [0, n)
constexpr int kDbgLossColWrite = 6;  // transposed CSR over the loss columns: a write position outside the row

// Bounds a caller knows about the operands of one sparse product; -1 = not known, not checked.
struct SpmmBounds {
  int64_t mat_rows = -1;  // rows of the CSR (length of rowptr minus one)
  int64_t src_rows = -1;  // rows of the gathered matrix
  int64_t nnz = -1;       // stored entries
};

#if defined(GCNSA_DEBUG) && defined(__CUDACC__)
#define GCNSA_DBG 1
// One status word per translation unit: device symbols do not cross translation units without relocatable
// device code, which this library is not built with.
#define GCNSA_DBG_WORD(name) static __device__ unsigned long long name = 0ull
__device__ __forceinline__ bool dbg_in(unsigned long long* word, long long v, long long lo, long long hi, int code) {
  if (v >= lo && v < hi) return true;
  atomicCAS(word, 0ull, ((unsigned long long)code << 56) | ((unsigned long long)v & 0x00ffffffffffffffull));
  return false;
}
#else
#define GCNSA_DBG 0
#endif

// Host side, one reader per translation unit that has a word (0 when the checks are compiled out).
int debug_word_spmm(unsigned long long* out, bool clear);
int debug_word_build(unsigned long long* out, bool clear);

}  // namespace gcnsa
