/*
 * CPU checker ("oracle") for subgraph-approximation GCN training.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 / int64, written from the paper
 * to be checked against it by eye.  It shares no code with the CUDA library
 * and must never be linked, imported or called by it; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * What is here (the sparse / graph steps; the dense steps live in oracle.py):
 *   key        - the 64-bit selection key that realises the random draw of Algorithm 1
 *   partition  - seeded stand-in for the METIS step of Section 4
 *   sample     - Algorithm 1, one (p, op) pair, breadth-first levels
 *   induced    - the augmented partition graph of Section 3.1 / Section 4 with
 *                self-loops and D^-1/2 (A+I) D^-1/2 weights (Section 4.1 footnote)
 *   transpose  - CSR -> CSR of the transpose
 *   spmm       - Y = A X, row by row, the definition
 *   neighbor sample - the fixed-size neighbour sample of the GraphSAGE variant
 *                (Section 4.1), drawn with the same selection key
 *
 * Every function returns 0 on success and a negative number on bad input.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

typedef int64_t i64;
typedef uint64_t u64;

/* ------------------------------------------------------------------ key --- */
/* Finalizer of SplitMix64 (Steele, Lea, Flood 2014): a bijection on 64 bits. */
static u64 mix64(u64 z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
  z ^= z >> 27; z *= 0x94D049BB133111EBULL;
  z ^= z >> 31;
  return z;
}

/* key(seed; w0..w3; v): absorb the words one at a time, the vertex id last.
 * For fixed (seed, w) the map v -> key is a bijection, so keys never tie and
 * "the nts smallest keys of a set" is a uniform random nts-subset that does
 * not depend on the order the set is visited in. */
u64 gcnsa_o_key(u64 seed, u64 w0, u64 w1, u64 w2, u64 w3, u64 v) {
  u64 h = mix64(seed);
  h = mix64(h ^ w0);
  h = mix64(h ^ w1);
  h = mix64(h ^ w2);
  h = mix64(h ^ w3);
  return mix64(h ^ v);
}

#define TAG_PART 1ULL
#define TAG_SAMPLE 2ULL
#define TAG_NEIGHBOR 3ULL

typedef struct { u64 key; i64 v; } keyed;
static int cmp_keyed(const void* a, const void* b) {
  u64 x = ((const keyed*)a)->key, y = ((const keyed*)b)->key;
  return x < y ? -1 : (x > y ? 1 : 0);
}
static int cmp_i64(const void* a, const void* b) {
  i64 x = *(const i64*)a, y = *(const i64*)b;
  return x < y ? -1 : (x > y ? 1 : 0);
}

/* ------------------------------------------------------------ partition --- */
/* Section 4 asks for parts of about equal vertex counts (METIS there).
 * mode 0 (range): part[v] = floor(v M / N).
 * mode 1 (hash):  rank the vertices by key(seed; TAG_PART,0,0,0; v) and cut the
 *                 ranking with the same rule.
 * mode 2 (user):  copy the caller's assignment. */
int gcnsa_o_partition(i64 n, i64 m, int mode, u64 seed, const int32_t* user, int32_t* part) {
  if (n < 0 || m < 1) return -1;
  if (mode == 0) {
    for (i64 v = 0; v < n; ++v) part[v] = (int32_t)((v * m) / n);
  } else if (mode == 1) {
    keyed* k = (keyed*)malloc(sizeof(keyed) * (size_t)(n > 0 ? n : 1));
    if (!k) return -2;
    for (i64 v = 0; v < n; ++v) { k[v].key = gcnsa_o_key(seed, TAG_PART, 0, 0, 0, (u64)v); k[v].v = v; }
    qsort(k, (size_t)n, sizeof(keyed), cmp_keyed);
    for (i64 r = 0; r < n; ++r) part[k[r].v] = (int32_t)((r * m) / n);
    free(k);
  } else if (mode == 2) {
    if (!user) return -1;
    for (i64 v = 0; v < n; ++v) {
      if (user[v] < 0 || user[v] >= m) return -3;
      part[v] = user[v];
    }
  } else {
    return -1;
  }
  return 0;
}

/* ---------------------------------------------------------- Algorithm 1 --- */
/* Algorithm 1 (Section 3.1) for one ordered pair (p, op), read as a walk over
 * breadth-first levels inside op:
 *   level 1 = the vertices of op that have a neighbour in p;
 *   level k + 1 = the vertices of op next to level k that are in no earlier level.
 * `want` vertices are still to be taken.  A level that holds fewer than `want`
 * vertices is taken whole and the walk moves one hop further; the first level
 * that holds at least `want` vertices supplies a uniform random subset of that
 * size (the `want` smallest selection keys) and ends the walk, as does an
 * empty level.  The paper states this recursively; the loop below takes the
 * same decisions in the same order.
 *
 * mark[v]: 0 = not seen, 1 = member of an earlier level, 2 = member of the
 * level being looked at. */

/* Collects the unseen vertices of op adjacent to `from[0..n_from)` into `out`
 * and marks them 2.  Returns how many. */
static i64 next_level(i64 n_from, const i64* from, const i64* rowptr, const int32_t* col, const int32_t* part,
                      int op, unsigned char* mark, i64* out) {
  i64 cnt = 0;
  for (i64 s = 0; s < n_from; ++s) {
    const i64 v = from[s];
    for (i64 e = rowptr[v]; e < rowptr[v + 1]; ++e) {
      const i64 u = col[e];
      if (part[u] == op && mark[u] == 0) { mark[u] = 2; out[cnt++] = u; }
    }
  }
  return cnt;
}

/* halo_out has room for nts entries and receives the selected vertices in
 * ascending id; returns their number, or a negative error.  depth_out
 * (nullable) = number of levels that contributed. */
i64 gcnsa_o_sample(i64 n, const i64* rowptr, const int32_t* col, const int32_t* part,
                   int p, int op, i64 nts, u64 seed, i64* halo_out, int32_t* depth_out) {
  if (depth_out) *depth_out = 0;
  if (p == op) return -1;
  if (nts <= 0 || n == 0) return 0;
  unsigned char* mark = (unsigned char*)calloc((size_t)n, 1);
  i64* cur = (i64*)malloc(sizeof(i64) * (size_t)n);
  i64* nxt = (i64*)malloc(sizeof(i64) * (size_t)n);
  keyed* kk = (keyed*)malloc(sizeof(keyed) * (size_t)n);
  if (!mark || !cur || !nxt || !kk) { free(mark); free(cur); free(nxt); free(kk); return -2; }

  /* level 1: the sources are the vertices of the original partition p */
  i64 n_own = 0;
  for (i64 v = 0; v < n; ++v) if (part[v] == p) nxt[n_own++] = v;
  i64 n_cur = next_level(n_own, nxt, rowptr, col, part, op, mark, cur);

  i64 want = nts, n_taken = 0;
  int k = 0;
  while (want > 0 && n_cur > 0) {
    ++k;
    if (n_cur >= want) {
      /* the last contributing level: a random subset of it, `want` vertices */
      for (i64 i = 0; i < n_cur; ++i) {
        kk[i].v = cur[i];
        kk[i].key = gcnsa_o_key(seed, TAG_SAMPLE, (u64)p, (u64)op, (u64)k, (u64)cur[i]);
      }
      qsort(kk, (size_t)n_cur, sizeof(keyed), cmp_keyed);
      for (i64 i = 0; i < want; ++i) halo_out[n_taken++] = kk[i].v;
      want = 0;
    } else {
      /* the whole level, then one hop further inside op */
      for (i64 i = 0; i < n_cur; ++i) { halo_out[n_taken++] = cur[i]; mark[cur[i]] = 1; }
      want -= n_cur;
      const i64 n_nxt = next_level(n_cur, cur, rowptr, col, part, op, mark, nxt);
      i64* t = cur; cur = nxt; nxt = t;
      n_cur = n_nxt;
    }
  }
  free(mark); free(cur); free(nxt); free(kk);
  qsort(halo_out, (size_t)n_taken, sizeof(i64), cmp_i64);
  if (depth_out) *depth_out = k;
  return n_taken;
}

/* nts = floor(O N_p / (M - 1)) with O in parts per million (Algorithm 1). */
i64 gcnsa_o_nts(i64 n_p, i64 m, i64 overlap_ppm) {
  if (m <= 1) return 0;
  return (i64)(((__int128)overlap_ppm * (__int128)n_p) / ((__int128)1000000 * (__int128)(m - 1)));
}

/* ------------------------------------------------ augmented partition graph */
/* members[0..n_loc): P_o[p] in local order (owned ascending, then halo
 * ascending).  The graph is the subgraph of G induced on these vertices plus a
 * self-loop on each (A + I).  Pass 1 (col_out == NULL) fills rowptr_out only;
 * pass 2 fills col_out (ascending in each row) and val_out = 1/sqrt(d_i d_j)
 * with d = row length including the self-loop. */
int gcnsa_o_induced(i64 n, const i64* rowptr, const int32_t* col, const i64* members, i64 n_loc,
                    i64* rowptr_out, i64* col_out, double* val_out) {
  i64* loc = (i64*)malloc(sizeof(i64) * (size_t)(n > 0 ? n : 1));
  if (!loc) return -2;
  for (i64 v = 0; v < n; ++v) loc[v] = -1;
  for (i64 i = 0; i < n_loc; ++i) {
    if (members[i] < 0 || members[i] >= n || loc[members[i]] != -1) { free(loc); return -1; }
    loc[members[i]] = i;
  }
  rowptr_out[0] = 0;
  for (i64 i = 0; i < n_loc; ++i) {
    i64 g = members[i], d = 1;                      /* the self-loop */
    for (i64 e = rowptr[g]; e < rowptr[g + 1]; ++e) if (loc[col[e]] >= 0) ++d;
    rowptr_out[i + 1] = rowptr_out[i] + d;
  }
  if (col_out) {
    for (i64 i = 0; i < n_loc; ++i) {
      i64 g = members[i], w = rowptr_out[i];
      col_out[w++] = i;
      for (i64 e = rowptr[g]; e < rowptr[g + 1]; ++e) if (loc[col[e]] >= 0) col_out[w++] = loc[col[e]];
      qsort(col_out + rowptr_out[i], (size_t)(w - rowptr_out[i]), sizeof(i64), cmp_i64);
    }
    if (val_out) {
      for (i64 i = 0; i < n_loc; ++i) {
        double di = (double)(rowptr_out[i + 1] - rowptr_out[i]);
        for (i64 e = rowptr_out[i]; e < rowptr_out[i + 1]; ++e) {
          i64 j = col_out[e];
          double dj = (double)(rowptr_out[j + 1] - rowptr_out[j]);
          val_out[e] = 1.0 / sqrt(di * dj);
        }
      }
    }
  }
  free(loc);
  return 0;
}

/* ------------------------------------------------------------ transpose --- */
/* B = A^T for an n_rows x n_cols CSR matrix; rows of B keep ascending columns. */
int gcnsa_o_transpose(i64 n_rows, i64 n_cols, const i64* rowptr, const i64* col, const double* val,
                      i64* t_rowptr, i64* t_col, double* t_val) {
  for (i64 j = 0; j <= n_cols; ++j) t_rowptr[j] = 0;
  for (i64 e = 0; e < rowptr[n_rows]; ++e) {
    if (col[e] < 0 || col[e] >= n_cols) return -1;
    t_rowptr[col[e] + 1]++;
  }
  for (i64 j = 0; j < n_cols; ++j) t_rowptr[j + 1] += t_rowptr[j];
  i64* fill = (i64*)malloc(sizeof(i64) * (size_t)(n_cols > 0 ? n_cols : 1));
  if (!fill) return -2;
  for (i64 j = 0; j < n_cols; ++j) fill[j] = t_rowptr[j];
  for (i64 i = 0; i < n_rows; ++i)
    for (i64 e = rowptr[i]; e < rowptr[i + 1]; ++e) {
      i64 w = fill[col[e]]++;
      t_col[w] = i;
      t_val[w] = val[e];
    }
  free(fill);
  return 0;
}

/* ----------------------------------------------------------------- spmm --- */
/* Y[i, :] = sum_e val[e] * X[col[e], :], row-major with leading dimension f. */
int gcnsa_o_spmm(i64 n_rows, const i64* rowptr, const i64* col, const double* val,
                 const double* x, i64 f, double* y) {
#pragma omp parallel for schedule(dynamic, 64)
  for (i64 i = 0; i < n_rows; ++i) {
    double* yi = y + i * f;
    for (i64 c = 0; c < f; ++c) yi[c] = 0.0;
    for (i64 e = rowptr[i]; e < rowptr[i + 1]; ++e) {
      const double a = val[e];
      const double* xj = x + col[e] * f;
      for (i64 c = 0; c < f; ++c) yi[c] += a * xj[c];
    }
  }
  return 0;
}

/* ------------------------------------------------------ input validation --- */
/* The method is stated for an undirected simple graph (Section 1 speaks of
 * bidirectional edges): 0 if the CSR is symmetric with no loops or repeats,
 * -4 not symmetric, -5 loop or repeat, -1 malformed. */
int gcnsa_o_validate(i64 n, const i64* rowptr, const int32_t* col) {
  if (rowptr[0] != 0) return -1;
  for (i64 v = 0; v < n; ++v) {
    if (rowptr[v + 1] < rowptr[v]) return -1;
    for (i64 e = rowptr[v]; e < rowptr[v + 1]; ++e) {
      i64 u = col[e];
      if (u < 0 || u >= n) return -1;
      if (u == v) return -5;
      for (i64 e2 = rowptr[v]; e2 < e; ++e2) if (col[e2] == u) return -5;
      int found = 0;
      for (i64 e2 = rowptr[u]; e2 < rowptr[u + 1]; ++e2) if (col[e2] == v) { found = 1; break; }
      if (!found) return -4;
    }
  }
  return 0;
}

/* ------------------------------------------- GraphSAGE neighbour sampling --- */
/* Section 4.1, GraphSAGE step 1: "a fixed number of neighbors" of a vertex is
 * sampled.  Read as: uniformly without replacement from the neighbours the
 * vertex has inside its extended partition (the vertex itself excluded); a
 * vertex with at most r neighbours keeps them all.  The draw is the r smallest
 * keys key(seed; TAG_NEIGHBOR, p, epoch * 256 + layer, v; u) over the neighbours
 * u, so it depends on (seed, p, epoch, layer, v) only.
 *
 * rowptr / col: CSR of the extended partition (A + I, local ids; the self-loop
 * is skipped here).  vs[0..n_v): local vertex ids, -1 = no vertex (count 0).
 * out: [n_v x r], row i receives the sample of vs[i] in ascending local id, the
 * rest of the row is -1; cnt[i] = its size.  Returns 0 or a negative error. */
int gcnsa_o_sample_neighbors(i64 n_loc, const i64* rowptr, const i64* col, u64 seed, u64 p, u64 epoch, u64 layer,
                             i64 n_v, const i64* vs, i64 r, i64* out, i64* cnt) {
  if (r < 0 || layer > 255) return -1;
  i64 max_deg = 1;
  for (i64 i = 0; i < n_loc; ++i) if (rowptr[i + 1] - rowptr[i] > max_deg) max_deg = rowptr[i + 1] - rowptr[i];
  keyed* kk = (keyed*)malloc(sizeof(keyed) * (size_t)max_deg);
  if (!kk) return -2;
  for (i64 i = 0; i < n_v; ++i) {
    i64* row = out + i * r;
    for (i64 s = 0; s < r; ++s) row[s] = -1;
    cnt[i] = 0;
    const i64 v = vs[i];
    if (v < 0) continue;
    if (v >= n_loc) { free(kk); return -1; }
    i64 deg = 0;
    for (i64 e = rowptr[v]; e < rowptr[v + 1]; ++e) {
      const i64 u = col[e];
      if (u == v) continue;
      kk[deg].v = u;
      kk[deg].key = gcnsa_o_key(seed, TAG_NEIGHBOR, p, epoch * 256 + layer, (u64)v, (u64)u);
      ++deg;
    }
    i64 take = deg;
    if (deg > r) {
      qsort(kk, (size_t)deg, sizeof(keyed), cmp_keyed);
      take = r;
    }
    for (i64 s = 0; s < take; ++s) row[s] = kk[s].v;
    qsort(row, (size_t)take, sizeof(i64), cmp_i64);
    cnt[i] = take;
  }
  free(kk);
  return 0;
}
