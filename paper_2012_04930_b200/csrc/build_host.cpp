// Host side of gcnsa_build_partitions: partition assignment, Algorithm 1 and the
// structure of every extended partition (CSR, transposed CSR, processing order).
// This is the master's one-time step of Section 3.2; values are computed on the
// device afterwards.
#include <algorithm>
#include <atomic>
#include <numeric>
#include <thread>

#include "internal.h"
#include "parts.h"

namespace gcnsa {

namespace {

inline uint64_t mix64(uint64_t z) {  // SplitMix64 finalizer (Steele, Lea, Flood 2014)
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

constexpr uint64_t kTagPart = 1, kTagSample = 2;

template <class F>
void parallel_for(int64_t n_items, int max_threads, F&& body) {
  int hw = (int)std::thread::hardware_concurrency();
  int nt = (int)std::max<int64_t>(1, std::min<int64_t>(std::min(hw > 0 ? hw : 4, max_threads), n_items));
  if (nt == 1) {
    for (int64_t i = 0; i < n_items; ++i) body(i);
    return;
  }
  std::atomic<int64_t> next{0};
  std::vector<std::thread> th;
  for (int t = 0; t < nt; ++t)
    th.emplace_back([&] {
      for (;;) {
        int64_t i = next.fetch_add(1);
        if (i >= n_items) break;
        body(i);
      }
    });
  for (auto& t : th) t.join();
}

struct Keyed {
  uint64_t key;
  int64_t v;
  bool operator<(const Keyed& o) const { return key < o.key; }
};

// Checks that the CSR is a simple undirected graph with ascending rows.
int validate(const gcnsa_graph* g) {
  const int64_t n = g->n;
  const int64_t* rp = g->rowptr;
  const int32_t* col = g->col;
  if (rp[0] != 0 || rp[n] != g->nnz) return fail(GCNSA_ERR_ARG, "rowptr[0] != 0 or rowptr[n] != nnz");
  const int64_t chunk = 4096, n_chunks = (n + chunk - 1) / chunk;
  std::atomic<int> status{0};
  parallel_for(n_chunks, 64, [&](int64_t ci) {
    if (status.load(std::memory_order_relaxed) != 0) return;
    for (int64_t v = ci * chunk; v < std::min(n, (ci + 1) * chunk); ++v) {
      if (rp[v + 1] < rp[v] || rp[v + 1] > g->nnz) { status = GCNSA_ERR_ARG; return; }
      for (int64_t e = rp[v]; e < rp[v + 1]; ++e) {
        const int64_t u = col[e];
        if (u < 0 || u >= n) { status = GCNSA_ERR_ARG; return; }
        if (u == v) { status = GCNSA_ERR_SELF_LOOP_OR_DUP; return; }
        if (e > rp[v]) {
          if (col[e - 1] == u) { status = GCNSA_ERR_SELF_LOOP_OR_DUP; return; }
          if (col[e - 1] > u) { status = GCNSA_ERR_ARG; return; }
        }
      }
    }
  });
  if (status != 0) return fail(status, "graph rows must be in range, ascending, without loops or repeats");
  // symmetry: v must appear in the (ascending, already checked) row of each neighbour
  parallel_for(n_chunks, 64, [&](int64_t ci) {
    if (status.load(std::memory_order_relaxed) != 0) return;
    for (int64_t v = ci * chunk; v < std::min(n, (ci + 1) * chunk); ++v)
      for (int64_t e = rp[v]; e < rp[v + 1]; ++e) {
        const int64_t u = col[e];
        if (!std::binary_search(col + rp[u], col + rp[u + 1], (int32_t)v)) { status = GCNSA_ERR_NOT_SYMMETRIC; return; }
      }
  });
  if (status != 0) return fail(status, "edge (u,v) present without (v,u)");
  return GCNSA_OK;
}

int assign(const gcnsa_graph* g, const gcnsa_part_opts* o, std::vector<int32_t>& part) {
  const int64_t n = g->n, m = o->m;
  part.resize((size_t)n);
  if (o->part_mode == GCNSA_PART_RANGE) {
    for (int64_t v = 0; v < n; ++v) part[v] = (int32_t)((v * m) / n);
  } else if (o->part_mode == GCNSA_PART_HASH) {
    std::vector<Keyed> k((size_t)n);
    for (int64_t v = 0; v < n; ++v) k[v] = {selection_key(o->seed, kTagPart, 0, 0, 0, (uint64_t)v), v};
    std::sort(k.begin(), k.end());
    for (int64_t r = 0; r < n; ++r) part[k[r].v] = (int32_t)((r * m) / n);
  } else if (o->part_mode == GCNSA_PART_USER) {
    if (!o->user_part) return fail(GCNSA_ERR_ARG, "user_part is NULL");
    for (int64_t v = 0; v < n; ++v) {
      if (o->user_part[v] < 0 || o->user_part[v] >= m) return fail(GCNSA_ERR_LABEL_RANGE, "user_part outside [0, m)");
      part[v] = o->user_part[v];
    }
  } else {
    return fail(GCNSA_ERR_ARG, "unknown part_mode");
  }
  return GCNSA_OK;
}

// Algorithm 1 for one partition p against every other partition, then the
// induced structure.  `mark` and `g2l` are scratch arrays of n entries.
int build_one(const gcnsa_graph* g, const gcnsa_part_opts* o, const std::vector<int32_t>& part, int32_t p,
              HostPart& hp) {
  const int64_t n = g->n;
  const int32_t m = o->m;
  const int64_t* rp = g->rowptr;
  const int32_t* col = g->col;
  std::vector<int64_t>& mem = hp.members;
  mem.clear();
  for (int64_t v = 0; v < n; ++v)
    if (part[v] == p) mem.push_back(v);
  hp.n_owned = (int64_t)mem.size();
  hp.nts = m > 1 ? (int64_t)(((unsigned __int128)o->overlap_ppm * (unsigned __int128)hp.n_owned) /
                             ((unsigned __int128)1000000 * (unsigned __int128)(m - 1)))
                 : 0;
  hp.depth.assign((size_t)m, 0);
  hp.max_depth = 0;
  std::vector<int64_t> halo;
  if (hp.nts > 0) {
    std::vector<uint8_t> mark((size_t)n, 0);
    // first level toward every other partition in one sweep over the cut edges
    std::vector<std::vector<int64_t>> level((size_t)m);
    for (int64_t i = 0; i < hp.n_owned; ++i) {
      const int64_t v = mem[i];
      for (int64_t e = rp[v]; e < rp[v + 1]; ++e) {
        const int32_t u = col[e];
        const int32_t q = part[u];
        if (q != p && !mark[u]) { mark[u] = 1; level[q].push_back(u); }
      }
    }
    std::vector<int64_t> next;
    std::vector<Keyed> keyed;
    for (int32_t op = 0; op < m; ++op) {
      if (op == p) continue;
      std::vector<int64_t>& cur = level[op];
      int64_t need = hp.nts;
      int32_t k = 1;
      while (need > 0 && !cur.empty()) {
        hp.depth[op] = k;
        if ((int64_t)cur.size() >= need) {
          keyed.resize(cur.size());
          for (size_t i = 0; i < cur.size(); ++i)
            keyed[i] = {selection_key(o->seed, kTagSample, (uint64_t)p, (uint64_t)op, (uint64_t)k, (uint64_t)cur[i]), cur[i]};
          if ((int64_t)keyed.size() > need) std::nth_element(keyed.begin(), keyed.begin() + need, keyed.end());
          for (int64_t i = 0; i < need; ++i) halo.push_back(keyed[i].v);
          need = 0;
        } else {
          halo.insert(halo.end(), cur.begin(), cur.end());
          need -= (int64_t)cur.size();
          next.clear();
          for (int64_t u : cur)
            for (int64_t e = rp[u]; e < rp[u + 1]; ++e) {
              const int32_t w = col[e];
              if (part[w] == op && !mark[w]) { mark[w] = 1; next.push_back(w); }
            }
          cur.swap(next);
          ++k;
        }
      }
      hp.max_depth = std::max(hp.max_depth, hp.depth[op]);
    }
    std::sort(halo.begin(), halo.end());
  }
  hp.n_halo = (int64_t)halo.size();
  mem.insert(mem.end(), halo.begin(), halo.end());
  hp.n = (int64_t)mem.size();
  if (hp.n >= (int64_t)INT32_MAX) return fail(GCNSA_ERR_TOO_LARGE, "extended partition has 2^31 rows or more");

  // induced structure: owned ids ascend with the global id and so do the sampled
  // ids, and every sampled id is larger than every owned one, so a row is
  // [owned neighbours asc.] ++ [sampled neighbours asc.] with the self-loop merged in.
  std::vector<int32_t> g2l((size_t)n, -1);
  for (int64_t i = 0; i < hp.n; ++i) g2l[mem[i]] = (int32_t)i;
  hp.rowptr.assign((size_t)hp.n + 1, 0);
  int64_t total = 0;
  for (int64_t i = 0; i < hp.n; ++i) {
    const int64_t v = mem[i];
    int64_t d = 1;
    for (int64_t e = rp[v]; e < rp[v + 1]; ++e) d += g2l[col[e]] >= 0;
    total += d;
    if (total >= (int64_t)INT32_MAX) return fail(GCNSA_ERR_TOO_LARGE, "extended partition has 2^31 non-zeros or more");
    hp.rowptr[i + 1] = (int32_t)total;
  }
  hp.nnz = total;
  hp.col.resize((size_t)total);
  for (int64_t i = 0; i < hp.n; ++i) {
    const int64_t v = mem[i];
    int32_t* w = hp.col.data() + hp.rowptr[i];
    const bool self_owned = i < hp.n_owned;
    bool self_done = false;
    for (int pass = 0; pass < 2; ++pass) {  // 0: owned neighbours, 1: sampled neighbours
      const bool self_here = (pass == 0) == self_owned;
      for (int64_t e = rp[v]; e < rp[v + 1]; ++e) {
        const int32_t l = g2l[col[e]];
        if (l < 0 || (l < hp.n_owned) != (pass == 0)) continue;
        if (self_here && !self_done && l > i) { *w++ = (int32_t)i; self_done = true; }
        *w++ = l;
      }
      if (self_here && !self_done) { *w++ = (int32_t)i; self_done = true; }
    }
  }
  // transposed structure by counting sort (a real transpose, nothing assumed)
  hp.t_rowptr.assign((size_t)hp.n + 1, 0);
  for (int64_t e = 0; e < total; ++e) hp.t_rowptr[hp.col[e] + 1]++;
  for (int64_t j = 0; j < hp.n; ++j) hp.t_rowptr[j + 1] += hp.t_rowptr[j];
  hp.t_col.resize((size_t)total);
  {
    std::vector<int32_t> fill(hp.t_rowptr.begin(), hp.t_rowptr.end() - 1);
    for (int64_t i = 0; i < hp.n; ++i)
      for (int32_t e = hp.rowptr[i]; e < hp.rowptr[i + 1]; ++e) hp.t_col[fill[hp.col[e]]++] = (int32_t)i;
  }
  // processing order: hub rows, then the others window by window, by descending length class inside a window, ties
  // by row index (order_key)
  const int64_t window = order_window_rows(o->order_window, hp.n);
  auto make_order = [&](const std::vector<int32_t>& rptr, int64_t thr, std::vector<int32_t>& ord) {
    ord.resize((size_t)hp.n);
    std::iota(ord.begin(), ord.end(), 0);
    std::vector<uint32_t> key((size_t)hp.n);
    for (int64_t i = 0; i < hp.n; ++i) key[i] = order_key(rptr[i + 1] - rptr[i], thr, hp.n, i, window);
    std::stable_sort(ord.begin(), ord.end(), [&](int32_t a, int32_t b) { return key[a] < key[b]; });
  };
  make_order(hp.rowptr, long_row_threshold(hp.nnz), hp.order);
  make_order(hp.t_rowptr, long_row_threshold(hp.nnz), hp.t_order);
  auto count_long = [&](const std::vector<int32_t>& rptr, const std::vector<int32_t>& ord) {
    int64_t k = 0;
    while (k < hp.n && rptr[ord[k] + 1] - rptr[ord[k]] >= long_row_threshold(hp.nnz)) ++k;
    return k;
  };
  hp.n_long = count_long(hp.rowptr, hp.order);
  hp.t_n_long = count_long(hp.t_rowptr, hp.t_order);
  hp.n_train = 0;
  const int64_t lim = o->loss_on_halo ? hp.n : hp.n_owned;
  std::vector<uint8_t> carries((size_t)hp.n, 0);
  for (int64_t i = 0; i < lim; ++i) {
    carries[i] = g->train_mask[mem[i]] != 0;
    hp.n_train += carries[i];
  }
  // the rows that carry loss, longest first (the last layer's forward product needs no others)
  hp.m_order.clear();
  hp.m_n_long = 0;
  hp.m_nnz = 0;
  {
    const int64_t thr = long_row_threshold(hp.nnz);
    for (int64_t k = 0; k < hp.n; ++k) {
      const int32_t r = hp.order[k];
      if (!carries[r]) continue;
      if (hp.rowptr[r + 1] - hp.rowptr[r] >= thr) hp.m_n_long = (int64_t)hp.m_order.size() + 1;
      hp.m_order.push_back(r);
      hp.m_nnz += hp.rowptr[r + 1] - hp.rowptr[r];
    }
  }
  // transposed structure restricted to the columns that carry loss
  hp.tm_rowptr.assign((size_t)hp.n + 1, 0);
  hp.tm_col.clear();
  hp.tm_col.reserve((size_t)total);
  for (int64_t j = 0; j < hp.n; ++j) {
    for (int32_t e = hp.t_rowptr[j]; e < hp.t_rowptr[j + 1]; ++e)
      if (carries[hp.t_col[e]]) hp.tm_col.push_back(hp.t_col[e]);
    hp.tm_rowptr[j + 1] = (int32_t)hp.tm_col.size();
  }
  make_order(hp.tm_rowptr, long_row_threshold((int64_t)hp.tm_col.size()), hp.tm_order);
  {
    int64_t k = 0;
    const int64_t thr = long_row_threshold((int64_t)hp.tm_col.size());
    while (k < hp.n && hp.tm_rowptr[hp.tm_order[k] + 1] - hp.tm_rowptr[hp.tm_order[k]] >= thr) ++k;
    hp.tm_n_long = k;
  }
  return GCNSA_OK;
}

}  // namespace

uint64_t selection_key(uint64_t seed, uint64_t w0, uint64_t w1, uint64_t w2, uint64_t w3, uint64_t v) {
  uint64_t h = mix64(seed);
  h = mix64(h ^ w0);
  h = mix64(h ^ w1);
  h = mix64(h ^ w2);
  h = mix64(h ^ w3);
  return mix64(h ^ v);
}

int check_build_args(const gcnsa_graph* g, const gcnsa_part_opts* o) {
  if (!g || !o) return fail(GCNSA_ERR_ARG, "NULL argument");
  if (g->n < 0 || g->nnz < 0 || (g->n > 0 && (!g->rowptr || !g->y || !g->train_mask || !g->x)) ||
      (g->nnz > 0 && !g->col))
    return fail(GCNSA_ERR_ARG, "graph arrays missing");
  if (g->f < 1 || g->c < 1 || g->ldx < g->f) return fail(GCNSA_ERR_ARG, "feature width, class count or ldx invalid");
  if (o->m < 1) return fail(GCNSA_ERR_ARG, "m < 1");
  if (g->n < o->m) return fail(GCNSA_ERR_ARG, "more partitions than vertices");
  if (g->n >= (int64_t)INT32_MAX) return fail(GCNSA_ERR_TOO_LARGE, "vertex ids must fit int32");
  if (o->order_window > 0 && o->order_window < kOrderWindowMin)
    return fail(GCNSA_ERR_ARG, "order_window must be 0 (default), negative (one window) or at least 256 rows");
  if (o->part_mode != GCNSA_PART_RANGE && o->part_mode != GCNSA_PART_HASH && o->part_mode != GCNSA_PART_USER)
    return fail(GCNSA_ERR_ARG, "unknown part_mode");
  if (o->part_mode == GCNSA_PART_USER && !o->user_part) return fail(GCNSA_ERR_ARG, "user_part is NULL");
  if (o->builder != GCNSA_BUILD_DEVICE && o->builder != GCNSA_BUILD_HOST) return fail(GCNSA_ERR_ARG, "unknown builder");
  return GCNSA_OK;
}

int validate_graph_host(const gcnsa_graph* g) {
  int rc = validate(g);
  if (rc) return rc;
  for (int64_t v = 0; v < g->n; ++v)
    if (g->y[v] < 0 || g->y[v] >= g->c) return fail(GCNSA_ERR_LABEL_RANGE, "label outside [0, c)");
  return GCNSA_OK;
}

int build_host(const gcnsa_graph* g, const gcnsa_part_opts* o, HostBuild* out) {
  if (!out) return fail(GCNSA_ERR_ARG, "NULL argument");
  int rc = check_build_args(g, o);
  if (rc) return rc;
  rc = validate_graph_host(g);
  if (rc) return rc;
  rc = assign(g, o, out->part);
  if (rc) return rc;
  out->parts.assign((size_t)o->m, HostPart());
  std::atomic<int> status{0};
  std::vector<std::string> msgs((size_t)o->m);
  parallel_for(o->m, 16, [&](int64_t p) {
    int r = build_one(g, o, out->part, (int32_t)p, out->parts[p]);
    if (r) { status = r; msgs[p] = gcnsa_last_error(); }
  });
  if (status != 0) {
    for (auto& s : msgs)
      if (!s.empty()) return fail(status, s);
    return fail(status, "partition build failed");
  }
  return GCNSA_OK;
}

}  // namespace gcnsa
