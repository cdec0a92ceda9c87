// Seeded synthetic inputs for the REST draft / verify path: token datastores,
// query contexts and a host suffix-array builder.  This file produces INPUT DATA
// only.  It contains none of the method's arithmetic (no retrieval, no trie, no
// selection, no attention, no acceptance) and is linked by neither the CUDA
// library nor the CPU oracle; both simply consume the arrays written here.
//
// Everything is a pure function of (seed, index) through a counter-based mixer,
// so any segment can be generated in parallel and regenerated identically.
//
// Build: g++ -O2 -fopenmp -shared -fPIC gen.cpp -o libdatagen.so
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <utility>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// splitmix64 finaliser (Steele, Lea, Flood 2014; Vigna's public-domain form).
inline uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
inline uint64_t h3(uint64_t seed, uint64_t stream, uint64_t a) {
  return mix64(mix64(seed ^ mix64(stream)) ^ a);
}
inline uint64_t h4(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
  return mix64(h3(seed, stream, a) ^ b);
}

enum Stream : uint64_t {
  S_SEG_INIT = 1, S_RANK = 2, S_TRANS = 3, S_SEG_KIND = 4, S_COPY = 5, S_UNIFORM = 6,
  S_CTX_KIND = 10, S_CTX_POS = 11, S_CTX_RANK = 12, S_CTX_INIT = 13, S_CTX_EDIT = 14,
  S_CTX_UNIFORM = 15
};

constexpr int SEG_LOG = 16;
constexpr int64_t SEG = int64_t(1) << SEG_LOG;
constexpr int MAX_R = 64;

// Integer CDF of Zipf(s) over ranks 1..R, as thresholds on a 32-bit uniform.
struct ZipfCdf {
  int R;
  uint32_t thr[MAX_R];
  ZipfCdf(double s, int R_) : R(R_) {
    double w[MAX_R], tot = 0;
    for (int r = 0; r < R; ++r) { w[r] = std::pow(double(r + 1), -s); tot += w[r]; }
    double acc = 0;
    for (int r = 0; r < R; ++r) {
      acc += w[r];
      double t = acc / tot * 4294967296.0;
      thr[r] = (r == R - 1 || t >= 4294967295.0) ? 0xFFFFFFFFu : uint32_t(t);
    }
  }
  int draw(uint32_t u) const {            // rank in 0..R-1
    int r = 0;
    while (r < R - 1 && u > thr[r]) ++r;
    return r;
  }
};

inline uint64_t state_hash(const int32_t* last, int order) {
  uint64_t s = 0x243F6A8885A308D3ull;
  for (int k = 0; k < order; ++k) s = mix64(s ^ uint64_t(uint32_t(last[k])));
  return s;
}

// Maps a hash to a token id with a power-law distribution over the vocabulary: id t has
// probability proportional to the integral of x^-1.3 over [t+1, t+2) (a truncated Pareto
// draw, floored).  Frequent ids make the chain's states recur, which is what gives the
// stream n-gram repetition; a uniform map would make nearly every state new.
constexpr double TOKEN_EXPONENT = 1.3;
inline int32_t heavy_tailed_token(uint64_t hsh, uint32_t vocab) {
  const double a = 1.0 - TOKEN_EXPONENT;                       // < 0
  double u = double(hsh >> 11) * (1.0 / 9007199254740992.0);   // [0,1)
  double top = std::pow(double(vocab) + 1.0, a);
  double x = std::pow(1.0 - u * (1.0 - top), 1.0 / a);         // in [1, vocab+1)
  int64_t id = int64_t(x) - 1;
  if (id < 0) id = 0;
  if (id >= int64_t(vocab)) id = int64_t(vocab) - 1;
  return int32_t(id);
}

// One Markov step: successor candidate `rank` of the state formed by the last `order` tokens.
inline int32_t successor(uint64_t seed, const int32_t* last, int order, int rank, uint32_t vocab) {
  return heavy_tailed_token(h4(seed, S_TRANS, state_hash(last, order), uint64_t(rank)), vocab);
}

struct ChainSpec { int order; uint32_t vocab; };

// Generates tokens [0,len) of one chain into out; `rank_stream`/`rank_base` select the
// rank draws, `init_stream`/`init_id` the first `order` tokens.
void run_chain(uint64_t seed, const ChainSpec& cs, const ZipfCdf& z, uint64_t rank_stream,
               uint64_t rank_base, uint64_t init_stream, uint64_t init_id, int64_t len,
               int32_t* out) {
  for (int64_t t = 0; t < len; ++t) {
    if (t < cs.order) {
      out[t] = heavy_tailed_token(h4(seed, init_stream, init_id, uint64_t(t)), cs.vocab);
    } else {
      int rank = z.draw(uint32_t(h3(seed, rank_stream, rank_base + uint64_t(t)) >> 32));
      out[t] = successor(seed, out + t - cs.order, cs.order, rank, cs.vocab);
    }
  }
}

}  // namespace

extern "C" {

uint64_t dg_mix(uint64_t seed, uint64_t stream, uint64_t a) { return h3(seed, stream, a); }

// Token stream of n tokens from an order-`order` Markov chain with Zipf(zipf_s)
// branching over R successor candidates, generated in independent 2^16-token segments.
//   copy_runs != 0 : overlay low-entropy copy runs (code-like repetition): at each
//                    position outside a run, with probability 1/64, replay 16..256
//                    tokens of the base stream from 2^8..2^20 positions earlier.
//   mixed != 0     : segment kinds alternate by hash: 1/4 uniform random tokens,
//                    3/8 low-entropy (Zipf 1.5 over 8 candidates), 3/8 the given chain.
void dg_markov_tokens(uint64_t seed, int64_t n, uint32_t vocab, int order, double zipf_s, int R,
                      int copy_runs, int mixed, int32_t* out) {
  if (R > MAX_R) R = MAX_R;
  ZipfCdf z(zipf_s, R), zlow(1.5, 8);
  ChainSpec cs{order, vocab};
  int64_t nseg = (n + SEG - 1) / SEG;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t g = 0; g < nseg; ++g) {
    int64_t base = g * SEG, len = std::min(SEG, n - base);
    int kind = 0;
    if (mixed) {
      uint64_t k = h3(seed, S_SEG_KIND, uint64_t(g)) & 7;
      kind = k < 2 ? 2 : (k < 5 ? 1 : 0);
    }
    if (kind == 2) {
      for (int64_t t = 0; t < len; ++t)
        out[base + t] = int32_t(h3(seed, S_UNIFORM, uint64_t(base + t)) % vocab);
    } else {
      run_chain(seed, cs, kind == 1 ? zlow : z, S_RANK, uint64_t(base), S_SEG_INIT, uint64_t(g),
                len, out + base);
    }
  }
  if (copy_runs) {
    std::vector<int32_t> basebuf(out, out + n);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t g = 0; g < nseg; ++g) {
      int64_t base = g * SEG, len = std::min(SEG, n - base);
      int64_t t = 0;
      while (t < len) {
        uint64_t r = h3(seed, S_COPY, uint64_t(base + t));
        if ((r & 63) == 0) {
          int64_t run = 16 + int64_t((r >> 8) % 241);
          int lg = 8 + int((r >> 20) % 13);
          int64_t off = (int64_t(1) << lg) + int64_t((r >> 28) % (uint64_t(1) << lg));
          int64_t src = base + t - off;
          if (src >= 0) {
            int64_t e = std::min(len, t + run);
            for (int64_t u = t; u < e; ++u) out[base + u] = basebuf[src + (u - t)];
            t = e;
            continue;
          }
        }
        ++t;
      }
    }
  }
}

// B query contexts of Lc tokens each (row-major [B, Lc]).  Kinds by hash of (seed, b):
//   70 % fresh samples of the same chain (same transitions, own rank stream);
//   20 % datastore slices whose token at distance d in [3,17] from the end is replaced
//        by a random token, so the longest matching suffix is about d-1;
//    5 % unmodified datastore slices; 5 % uniform random tokens.
void dg_contexts(uint64_t seed, const int32_t* tokens, int64_t n, uint32_t vocab, int order,
                 double zipf_s, int R, int32_t B, int32_t Lc, int32_t* out) {
  if (R > MAX_R) R = MAX_R;
  ZipfCdf z(zipf_s, R);
  ChainSpec cs{order, vocab};
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t b = 0; b < B; ++b) {
    int32_t* row = out + int64_t(b) * Lc;
    uint64_t kind = h3(seed, S_CTX_KIND, uint64_t(b)) % 100;
    bool can_slice = n >= Lc;
    if (kind < 70 || (!can_slice && kind < 95)) {
      run_chain(seed, cs, z, S_CTX_RANK, uint64_t(b) << 32, S_CTX_INIT, uint64_t(b), Lc, row);
    } else if (kind < 95) {
      int64_t pos = int64_t(h3(seed, S_CTX_POS, uint64_t(b)) % uint64_t(n - Lc + 1));
      std::memcpy(row, tokens + pos, sizeof(int32_t) * size_t(Lc));
      if (kind < 90) {
        uint64_t e = h3(seed, S_CTX_EDIT, uint64_t(b));
        int d = 3 + int(e % 15);
        if (d <= Lc) {
          int32_t old = row[Lc - d];
          int32_t nw = int32_t((e >> 16) % vocab);
          if (nw == old) nw = int32_t((uint32_t(nw) + 1u) % vocab);
          row[Lc - d] = nw;
        }
      }
    } else {
      for (int32_t t = 0; t < Lc; ++t)
        row[t] = int32_t(h4(seed, S_CTX_UNIFORM, uint64_t(b), uint64_t(t)) % vocab);
    }
  }
}

// ---------------------------------------------------------------------------------
// Host suffix-array builder (input preparation).
//
// Sorts suffix start positions by their first W tokens (a suffix that runs off the end
// of the stream sorts before any longer suffix it is a prefix of); suffixes that agree
// on all W tokens are ordered by start position.  W = 0 means "compare to the end",
// i.e. the true suffix array.  Method: bucket by first token, sort packed k-token keys
// inside the buckets, then prefix doubling restricted to still-tied groups.
// sa_bytes selects int32 (4) or int64 (8) output.  Returns 0 on success.
// ---------------------------------------------------------------------------------
int dg_build_sa(const int32_t* T, int64_t n, uint32_t vocab, int W, int sa_bytes, void* out) {
  if (n < 0 || (sa_bytes != 4 && sa_bytes != 8)) return 1;
  if (sa_bytes == 4 && n > int64_t(0x7FFFFFFF)) return 1;
  if (n == 0) return 0;
  using idx_t = int64_t;
  int bits = 1;
  while ((uint64_t(1) << bits) < uint64_t(vocab) + 1) ++bits;   // symbols 0..vocab (0 = end)
  int k = std::max(1, std::min(8, 64 / bits));                  // tokens per packed key
  auto key_at = [&](idx_t p) {
    uint64_t key = 0;
    for (int j = 0; j < k; ++j) {
      uint64_t sym = (p + j < n) ? uint64_t(uint32_t(T[p + j])) + 1 : 0;
      key = (key << bits) | sym;
    }
    return key;
  };

  std::vector<idx_t> sa(n);
  std::vector<uint64_t> keys(n);   // packed key of sa[j], in SA order
  {
    // Bucket by first token (counting sort), then sort (key, position) pairs per bucket.
    std::vector<idx_t> start(size_t(vocab) + 2, 0);
    for (idx_t i = 0; i < n; ++i) start[size_t(uint32_t(T[i])) + 1]++;
    for (size_t v = 1; v < start.size(); ++v) start[v] += start[v - 1];
    std::vector<idx_t> cur(start.begin(), start.end() - 1);
    for (idx_t i = 0; i < n; ++i) sa[cur[uint32_t(T[i])]++] = i;
    int64_t nb = int64_t(vocab);
#pragma omp parallel
    {
      std::vector<std::pair<uint64_t, idx_t>> buf;
#pragma omp for schedule(dynamic, 16)
      for (int64_t v = 0; v < nb; ++v) {
        idx_t s = start[v], e = start[v + 1];
        if (e - s < 2) {
          if (e > s) keys[s] = key_at(sa[s]);
          continue;
        }
        buf.resize(size_t(e - s));
        for (idx_t j = s; j < e; ++j) buf[j - s] = {key_at(sa[j]), sa[j]};
        std::sort(buf.begin(), buf.end());
        for (idx_t j = s; j < e; ++j) { sa[j] = buf[j - s].second; keys[j] = buf[j - s].first; }
      }
    }
  }

  // rank[p] = first SA slot of the group of suffixes equal to p's on the first h tokens.
  std::vector<idx_t> rank(n), nrank(n);
  std::vector<idx_t> gstart;   // starts of groups with more than one member
  std::vector<idx_t> gend;
  {
    idx_t s = 0;
    uint64_t ks = keys[0];
    for (idx_t j = 1; j <= n; ++j) {
      uint64_t kj = j < n ? keys[j] : 0;
      if (j == n || kj != ks) {
        for (idx_t u = s; u < j; ++u) rank[sa[u]] = s;
        if (j - s > 1) { gstart.push_back(s); gend.push_back(j); }
        s = j; ks = kj;
      }
    }
  }
  std::vector<uint64_t>().swap(keys);
  int64_t h = k;
  while (!gstart.empty() && (W == 0 ? h < n : h < W)) {
    int64_t ng = int64_t(gstart.size());
    std::vector<std::vector<idx_t>> ns_t, ne_t;
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    ns_t.resize(nthreads); ne_t.resize(nthreads);
    std::vector<std::vector<std::pair<idx_t, idx_t>>> changes(nthreads);  // (position, new rank)
#pragma omp parallel
    {
      int tid = 0;
#ifdef _OPENMP
      tid = omp_get_thread_num();
#endif
      std::vector<std::pair<idx_t, idx_t>> buf;
#pragma omp for schedule(dynamic, 64)
      for (int64_t g = 0; g < ng; ++g) {
        idx_t s = gstart[g], e = gend[g];
        buf.resize(size_t(e - s));
        for (idx_t j = s; j < e; ++j) {
          idx_t p = sa[j];
          buf[j - s] = {p + h < n ? rank[p + h] : idx_t(-1), p};
        }
        std::sort(buf.begin(), buf.end());   // ties keep ascending position
        idx_t sub = s;
        for (idx_t j = s; j < e; ++j) {
          sa[j] = buf[j - s].second;
          bool last = (j + 1 == e) || buf[j + 1 - s].first != buf[j - s].first;
          if (last) {
            if (sub != s || j + 1 != e)
              for (idx_t u = sub; u <= j; ++u) changes[tid].push_back({buf[u - s].second, sub});
            if (j + 1 - sub > 1) { ns_t[tid].push_back(sub); ne_t[tid].push_back(j + 1); }
            sub = j + 1;
          }
        }
      }
    }
    for (auto& c : changes) for (auto& pr : c) rank[pr.first] = pr.second;
    std::vector<std::pair<idx_t, idx_t>> groups;
    for (int t = 0; t < nthreads; ++t)
      for (size_t i = 0; i < ns_t[t].size(); ++i) groups.push_back({ns_t[t][i], ne_t[t][i]});
    std::sort(groups.begin(), groups.end());
    gstart.clear(); gend.clear();
    for (auto& g : groups) { gstart.push_back(g.first); gend.push_back(g.second); }
    h *= 2;
  }
  // Remaining ties (equal on >= W tokens): ascending start position.
  {
    int64_t ng = int64_t(gstart.size());
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t g = 0; g < ng; ++g) std::sort(sa.begin() + gstart[g], sa.begin() + gend[g]);
  }
  if (sa_bytes == 4) {
    int32_t* o = static_cast<int32_t*>(out);
    for (idx_t i = 0; i < n; ++i) o[i] = int32_t(sa[i]);
  } else {
    std::memcpy(out, sa.data(), sizeof(int64_t) * size_t(n));
  }
  return 0;
}

// Full check of a suffix array at any size: sa is a permutation of 0..n-1 and adjacent
// entries are ordered by their first W tokens (W = 0: whole suffixes; cost then depends
// on repeat lengths), ties in ascending position.  Returns 0 when valid, else a code
// (1 bad args, 2 out of range, 3 duplicate, 4 order violated, 5 tie order violated).
int dg_verify_sa(const int32_t* T, int64_t n, int W, int sa_bytes, const void* sa_) {
  if (sa_bytes != 4 && sa_bytes != 8) return 1;
  auto at = [&](int64_t i) -> int64_t {
    return sa_bytes == 4 ? int64_t(static_cast<const int32_t*>(sa_)[i])
                         : static_cast<const int64_t*>(sa_)[i];
  };
  std::vector<uint8_t> seen(size_t(n), 0);
  for (int64_t i = 0; i < n; ++i) {
    int64_t p = at(i);
    if (p < 0 || p >= n) return 2;
    if (seen[p]) return 3;
    seen[p] = 1;
  }
  int bad = 0;
#pragma omp parallel for schedule(static) reduction(max : bad)
  for (int64_t i = 1; i < n; ++i) {
    int64_t a = at(i - 1), b = at(i);
    int64_t lim = W == 0 ? n : W;
    int cmp = 0;   // -1 a<b, 0 tie, 1 a>b
    for (int64_t j = 0; j < lim; ++j) {
      bool ea = a + j >= n, eb = b + j >= n;
      if (ea || eb) { cmp = (ea && eb) ? 0 : (ea ? -1 : 1); break; }
      uint32_t ta = uint32_t(T[a + j]), tb = uint32_t(T[b + j]);
      if (ta != tb) { cmp = ta < tb ? -1 : 1; break; }
    }
    if (cmp > 0) bad = std::max(bad, 4);
    else if (cmp == 0 && a > b) bad = std::max(bad, 5);
  }
  return bad;
}

}  // extern "C"
