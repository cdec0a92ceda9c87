// CPU oracle for one REST decoding step (retrieval draft + tree verification).
//
// TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of
// the paper's definitions, used to check the CUDA library.  It shares no code with
// the CUDA path; nothing in the product may call it.  Only the tests, the smoke check
// and the benchmark's CPU-baseline leg load it.
//
// What follows the paper, function by function:
//   oracle_suffix_array   Sec. 3.2 "Retrieving from the datastore": exact match is served
//                         by a suffix array; here: std::sort of all suffixes.
//   oracle_retrieve       Algorithm 1: longest suffix of the context (n_max down to n_min)
//                         that occurs in the datastore; its range in the suffix array.
//   oracle_draft          Algorithm 1 + Algorithm 2 + Sec. 3.2 "Draft verification":
//                         continuations of the matches, a Trie (std::map keyed by prefix)
//                         whose node weight is the number of candidates with that prefix,
//                         the c = N heaviest nodes, the breadth-first pseudo sequence, its
//                         ancestor ("tree attention") mask and position ids.
//   oracle_tree_attention Sec. 3.2 "Draft verification": every draft token attends to the
//                         whole prefix and to its own ancestors; fp64 softmax attention.
//   oracle_accept         Sec. 3.2 "Draft acceptance": draft tokens are accepted from the
//                         root while they equal the verifier's token at that position.
//
// Readings taken where the paper is silent (stated again next to the code):
//   * the suffix-length loop stops at n_min (paper: loops while S is empty); no match at
//     any length gives an empty tree;
//   * at most K candidates are used: when more match, candidate j is the match at slot
//     lo + floor(j*cnt/K) of the suffix-array range (mode 0) or lo + j (mode 1);
//   * ties between equally heavy Trie nodes: shallower first, then the lexicographically
//     smaller token path;
//   * siblings in the breadth-first order ascend by token id; position id = context
//     length + depth - 1; the empty prefix is not a node.
//
// Pins (tests/test_oracle_*.py): brute-force substring scans on tiny datastores, a
// hand-worked example, Trie invariants, losslessness against token-by-token decoding,
// and for attention: an independent causal-attention routine over prefix + path, chain
// and star trees, constant-V and zero-K closed forms.
//
// Build: g++ -O2 -fopenmp -std=c++17 -shared -fPIC rest_oracle.cpp -o librest_oracle.so
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

struct SaView {
  const void* p;
  int bytes;
  int64_t operator[](int64_t i) const {
    return bytes == 4 ? int64_t(static_cast<const int32_t*>(p)[i])
                      : static_cast<const int64_t*>(p)[i];
  }
};

// Compares the first n tokens of the suffix starting at p with q[0..n).  Tokens compare as
// unsigned integers; a suffix that ends before a difference is found is the smaller one.
int cmp_suffix(const int32_t* T, int64_t n_tokens, int64_t p, const int32_t* q, int n) {
  for (int k = 0; k < n; ++k) {
    if (p + k >= n_tokens) return -1;
    uint32_t a = uint32_t(T[p + k]), b = uint32_t(q[k]);
    if (a != b) return a < b ? -1 : 1;
  }
  return 0;
}

// First slot whose suffix is >= q (strict=false) or > q (strict=true) on the first n tokens.
int64_t bound(const int32_t* T, int64_t n_tokens, const SaView& sa, const int32_t* q, int n,
              bool strict) {
  int64_t lo = 0, hi = n_tokens;
  while (lo < hi) {
    int64_t mid = lo + (hi - lo) / 2;
    int c = cmp_suffix(T, n_tokens, sa[mid], q, n);
    bool before = strict ? (c <= 0) : (c < 0);
    if (before) lo = mid + 1; else hi = mid;
  }
  return lo;
}

struct Match { int n; int64_t lo, hi; };

// Algorithm 1.  n starts at min(n_max, ctx_len) and decreases to n_min; the first length
// with a non-empty range wins.  {0,0,0} when nothing matches.
Match retrieve(const int32_t* T, int64_t n_tokens, const SaView& sa, const int32_t* ctx,
               int32_t ctx_len, int n_max, int n_min) {
  for (int n = std::min<int64_t>(n_max, ctx_len); n >= n_min && n >= 1; --n) {
    const int32_t* q = ctx + (ctx_len - n);
    int64_t lo = bound(T, n_tokens, sa, q, n, false);
    int64_t hi = bound(T, n_tokens, sa, q, n, true);
    if (hi > lo) return {n, lo, hi};
  }
  return {0, 0, 0};
}

inline double bf16_to_double(uint16_t b) {
  uint32_t u = uint32_t(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return double(f);
}

}  // namespace

extern "C" {

struct oracle_params { int32_t n_max, n_min, K, m, N, sample_mode; };

int oracle_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// True suffix array by comparison sort of whole suffixes (small inputs only).
int oracle_suffix_array(const int32_t* T, int64_t n, int64_t* sa) {
  std::iota(sa, sa + n, int64_t(0));
  std::sort(sa, sa + n, [&](int64_t a, int64_t b) {
    while (a < n && b < n) {
      uint32_t x = uint32_t(T[a]), y = uint32_t(T[b]);
      if (x != y) return x < y;
      ++a; ++b;
    }
    return a > b;   // the suffix that ran out first (started later) is the shorter one
  });
  return 0;
}

int oracle_retrieve(const int32_t* T, int64_t n_tokens, const void* sa_, int sa_bytes,
                    const int32_t* ctx, int32_t ctx_len, int n_max, int n_min,
                    int32_t* match_n, int64_t* lo, int64_t* hi) {
  SaView sa{sa_, sa_bytes};
  Match mt = retrieve(T, n_tokens, sa, ctx, ctx_len, n_max, n_min);
  *match_n = mt.n; *lo = mt.lo; *hi = mt.hi;
  return 0;
}

// One draft tree per context.  Outputs are [B,N] (mask [B,N,ceil(N/32)]); slots past
// n_nodes hold token -1, parent -1, depth 0, pos_id ctx_len, own mask bit, count 0.
// status[b]: 0 ok, 1 context token outside [0,vocab), 2 suffix-array entry out of range.
int oracle_draft(const int32_t* T, int64_t n_tokens, const void* sa_, int sa_bytes, uint32_t vocab,
                 const oracle_params* prm, const int32_t* ctx, int64_t ctx_stride,
                 const int32_t* ctx_len, int32_t B, int32_t* tokens, int32_t* parents,
                 int32_t* depth, int32_t* pos_ids, uint32_t* mask, int32_t* n_nodes,
                 int32_t* match_n, int64_t* match_range, int32_t* node_count, int32_t* status) {
  const int N = prm->N, m = prm->m, K = prm->K, Wm = (N + 31) / 32;
  SaView sa{sa_, sa_bytes};
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t b = 0; b < B; ++b) {
    const int32_t* s = ctx + int64_t(b) * ctx_stride;
    const int32_t len = ctx_len[b];
    int32_t* tok = tokens + int64_t(b) * N;
    int32_t* par = parents + int64_t(b) * N;
    int32_t* dep = depth + int64_t(b) * N;
    int32_t* pos = pos_ids + int64_t(b) * N;
    uint32_t* msk = mask + int64_t(b) * N * Wm;
    int32_t* cntout = node_count ? node_count + int64_t(b) * N : nullptr;
    for (int i = 0; i < N; ++i) {
      tok[i] = -1; par[i] = -1; dep[i] = 0; pos[i] = len;
      for (int w = 0; w < Wm; ++w) msk[int64_t(i) * Wm + w] = 0;
      msk[int64_t(i) * Wm + (i >> 5)] = 1u << (i & 31);
      if (cntout) cntout[i] = 0;
    }
    n_nodes[b] = 0; match_n[b] = 0; match_range[2 * b] = 0; match_range[2 * b + 1] = 0;
    status[b] = 0;

    bool bad_ctx = false;
    for (int k = 0; k < std::min<int32_t>(prm->n_max, len); ++k) {
      int32_t t = s[len - 1 - k];
      if (t < 0 || uint32_t(t) >= vocab) bad_ctx = true;
    }
    if (bad_ctx) { status[b] = 1; continue; }

    // Algorithm 1: candidates S = continuations of the longest matching suffix.
    Match mt = retrieve(T, n_tokens, sa, s, len, prm->n_max, prm->n_min);
    if (mt.n == 0) continue;
    int64_t cnt = mt.hi - mt.lo;
    int64_t Kp = std::min<int64_t>(cnt, K);
    std::vector<std::vector<int32_t>> S;
    bool bad_sa = false;
    for (int64_t j = 0; j < Kp; ++j) {
      int64_t slot = (cnt <= K || prm->sample_mode == 1) ? mt.lo + j
                     : mt.lo + int64_t((__int128(j) * cnt) / K);
      int64_t p = sa[slot];
      if (p < 0 || p >= n_tokens) { bad_sa = true; break; }
      std::vector<int32_t> t;
      for (int d = 0; d < m && p + mt.n + d < n_tokens; ++d) t.push_back(T[p + mt.n + d]);
      S.push_back(std::move(t));
    }
    if (bad_sa) { status[b] = 2; continue; }
    match_n[b] = mt.n; match_range[2 * b] = mt.lo; match_range[2 * b + 1] = mt.hi;

    // Algorithm 2, first loop: insert every non-empty prefix of every candidate.
    std::map<std::vector<int32_t>, int64_t> trie;
    for (const auto& t : S)
      for (size_t d = 1; d <= t.size(); ++d)
        trie[std::vector<int32_t>(t.begin(), t.begin() + d)] += 1;

    // Algorithm 2, second part: keep the c = N heaviest nodes.
    struct Node { int64_t w; std::vector<int32_t> path; };
    std::vector<Node> nodes;
    for (const auto& kv : trie) nodes.push_back({kv.second, kv.first});
    std::sort(nodes.begin(), nodes.end(), [](const Node& a, const Node& c) {
      if (a.w != c.w) return a.w > c.w;
      if (a.path.size() != c.path.size()) return a.path.size() < c.path.size();
      return a.path < c.path;
    });
    if (int64_t(nodes.size()) > N) nodes.resize(N);

    // Breadth-first pseudo sequence: by depth, then by path (siblings ascend by token).
    std::sort(nodes.begin(), nodes.end(), [](const Node& a, const Node& c) {
      if (a.path.size() != c.path.size()) return a.path.size() < c.path.size();
      return a.path < c.path;
    });
    std::map<std::vector<int32_t>, int> index_of;
    for (size_t i = 0; i < nodes.size(); ++i) index_of[nodes[i].path] = int(i);
    for (size_t i = 0; i < nodes.size(); ++i) {
      const auto& p = nodes[i].path;
      tok[i] = p.back();
      dep[i] = int32_t(p.size());
      pos[i] = len + int32_t(p.size()) - 1;
      if (cntout) cntout[i] = int32_t(nodes[i].w);
      if (p.size() > 1) {
        auto it = index_of.find(std::vector<int32_t>(p.begin(), p.end() - 1));
        par[i] = it == index_of.end() ? -2 : it->second;   // -2 would flag a non-closed set
      }
      // tree-attention mask: the node itself and every ancestor
      for (size_t d = 1; d <= p.size(); ++d) {
        auto it = index_of.find(std::vector<int32_t>(p.begin(), p.begin() + d));
        if (it != index_of.end())
          msk[int64_t(i) * Wm + (it->second >> 5)] |= 1u << (it->second & 31);
      }
    }
    n_nodes[b] = int32_t(nodes.size());
  }
  return 0;
}

// Tree attention in fp64.  q: bf16 bits [B,N,H,D]; k,v: bf16 bits [B,H_kv,*,D]; strides in
// elements: {q_b,q_n,q_h, kv_b,kv_h,kv_l, (unused x3)}; D contiguous.  Row i of context b
// attends keys 0..L-1 (L = kv_len[b]) and key L+j for every set bit j of its mask row.
// out: dense fp64 [B,N,H,D]; lse (optional): fp64 [B,H,N], natural log of the softmax sum
// of scaled scores.
int oracle_tree_attention(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                          const int64_t* strides, const int32_t* kv_len, const uint32_t* mask,
                          int32_t B, int32_t H, int32_t H_kv, int32_t N, int32_t D, double scale,
                          double* out, double* lse) {
  const int Wm = (N + 31) / 32;
  const int group = H / H_kv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int32_t b = 0; b < B; ++b) {
    for (int32_t h = 0; h < H; ++h) {
      const int64_t L = kv_len[b];
      const int hk = h / group;
      const uint16_t* kb = k + b * strides[3] + hk * strides[4];
      const uint16_t* vb = v + b * strides[3] + hk * strides[4];
      std::vector<double> sc(static_cast<size_t>(L + N)), qd(static_cast<size_t>(D)),
          acc(static_cast<size_t>(D));
      std::vector<int64_t> keys;
      for (int32_t i = 0; i < N; ++i) {
        const uint16_t* qi = q + b * strides[0] + i * strides[1] + h * strides[2];
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_double(qi[d]);
        keys.clear();
        for (int64_t j = 0; j < L; ++j) keys.push_back(j);
        const uint32_t* mrow = mask + (int64_t(b) * N + i) * Wm;
        for (int j = 0; j < N; ++j)
          if ((mrow[j >> 5] >> (j & 31)) & 1u) keys.push_back(L + j);
        double mx = -INFINITY;
        for (size_t t = 0; t < keys.size(); ++t) {
          const uint16_t* kr = kb + keys[t] * strides[5];
          double s = 0;
          for (int d = 0; d < D; ++d) s += qd[d] * bf16_to_double(kr[d]);
          sc[t] = s * scale;
          mx = std::max(mx, sc[t]);
        }
        double den = 0;
        for (size_t t = 0; t < keys.size(); ++t) { sc[t] = std::exp(sc[t] - mx); den += sc[t]; }
        std::fill(acc.begin(), acc.end(), 0.0);
        for (size_t t = 0; t < keys.size(); ++t) {
          const uint16_t* vr = vb + keys[t] * strides[5];
          double p = sc[t] / den;
          for (int d = 0; d < D; ++d) acc[d] += p * bf16_to_double(vr[d]);
        }
        double* o = out + ((int64_t(b) * N + i) * H + h) * D;
        for (int d = 0; d < D; ++d) o[d] = acc[d];
        if (lse) lse[(int64_t(b) * H + h) * N + i] = mx + std::log(den);
      }
    }
  }
  return 0;
}

// Draft acceptance.  verifier_tokens [B,N+1]: slot 0 is the verifier's token after the
// prefix, slot i+1 its token after draft node i.  Walk from the root: if the current node
// has a child whose token equals the verifier's token there, accept the child and go on
// from it; otherwise stop.  out_tokens = accepted tokens followed by the verifier's token
// at the stop (the token plain decoding would have produced); unused slots are -1.
int oracle_accept(const int32_t* tokens, const int32_t* parents, const int32_t* n_nodes,
                  const int32_t* verifier_tokens, int32_t B, int32_t N, int32_t max_depth,
                  int32_t* accept_len, int32_t* accept_nodes, int32_t* out_tokens) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t* tok = tokens + int64_t(b) * N;
    const int32_t* par = parents + int64_t(b) * N;
    const int32_t* ver = verifier_tokens + int64_t(b) * (N + 1);
    int32_t* an = accept_nodes + int64_t(b) * max_depth;
    int32_t* ot = out_tokens + int64_t(b) * (max_depth + 1);
    for (int d = 0; d < max_depth; ++d) an[d] = -1;
    for (int d = 0; d <= max_depth; ++d) ot[d] = -1;
    int cur = -1, len = 0;
    while (len < max_depth) {
      int32_t want = ver[cur + 1];
      int child = -1;
      for (int i = 0; i < n_nodes[b]; ++i)
        if (par[i] == cur && tok[i] == want) { child = i; break; }
      if (child < 0) break;
      an[len] = child; ot[len] = want; ++len; cur = child;
    }
    ot[len] = ver[cur + 1];
    accept_len[b] = len;
  }
  return 0;
}

}  // extern "C"
