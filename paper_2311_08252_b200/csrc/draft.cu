// rest_draft: Algorithm 1 (longest-suffix retrieval over a suffix array), Algorithm 2
// (Trie weights and the c heaviest nodes) and the breadth-first pseudo sequence with its
// ancestor mask (Sec. 3.2), one thread block per context, everything in one launch.
//
// Phases inside the block:
//   1 search   a warp per suffix length: the bucket index (when the datastore has one) gives the
//              suffix-array range of the query's first token pair, a 32-ary lower bound inside
//              it (every lane probes one slot per round, a ballot narrows the interval) finds
//              the first match, and for the longest length that matched a galloping + 32-ary
//              upper bound finds the end of the run.
//   2 gather   candidate rows in suffix-array order, which is also the lexicographic order of
//              the continuations.  A warp fetches its 32 rows (and the row before them) with
//              coalesced loads: lane l reads word l, 32 + l, ... of the rows laid end to end,
//              so a load touches three or four rows instead of 32, and the rows pass through
//              a shared-memory staging area.  Only the common-prefix length with the previous
//              row survives: for every depth d the bitmap "row j starts a new Trie node at
//              depth d" (lcp_j < d).
//   3 select   weight of node (d, j) = distance to the next set bit of bitmap d.  All passes
//              run over (depth, bitmap word) pairs, not over rows: two adjacent set bits are a
//              node of weight 1 (counted with one popcount per word), a set bit followed by a
//              clear one is a heavier node (visited one by one).  The N largest by (weight
//              desc, depth asc, row asc) come from a two-level radix histogram over (weight,
//              depth) and a prefix sum over the words of the tie depth.
//   4 emit     rank the kept nodes by (depth, row), look up parents through the bitmap of the
//              depth above, build ancestor masks, fetch the node tokens.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxM = REST_MAX_M;
constexpr int kMaxN = REST_MAX_N;
constexpr int kHistHi = 1056;   // bins of key >> 10, key < 2^20 + 32
constexpr int kHistLo = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;
// Batched path (calls with far more contexts than the GPU holds at once): threads per block,
// lanes per probe round once the probes leave L2, the number of 32-wide rounds before that,
// and whether the suffix lengths are searched in two steps.  Measured at 4096 contexts on a
// 100 M-token datastore: 512 threads, every length, 32 lanes 565 us; 256 threads with 4 or 8
// lanes 533 / 509 us; 256 threads, 8 lanes, two steps 474 us; 128 threads were slower again.
constexpr int kTpThreads = 256;
constexpr int kTpArity = 8;
constexpr bool kTpStaged = true;
constexpr int kWideRounds = 3;
// three-launch form: block sizes of the search and of the build of contexts with at most
// kLightRows candidates, and of the build of the others
constexpr int kSearchThreads = 128;
constexpr int kLightThreads = 128;
constexpr int kLightRows = 256;
// Blocks of contexts with long candidate lists: kThreads (two per SM by registers) unless the
// K cap is so large that shared memory allows only two blocks per SM anyway; then kBigThreads,
// which doubles the threads an SM gives to such a context (K = 20000, m = 16: 880 -> 415 us at
// 1024 contexts, 1670 -> 1181 us at 4096; at K = 5000 the same change loses 4-13 % in large calls).
constexpr int kBigThreads = 1024;
constexpr size_t kBigSmemBytes = 56 * 1024;

struct DraftArgs {
  const int32_t* T;
  const void* sa;
  int64_t n_tokens;
  uint32_t vocab;
  int n_max, n_min, K, m, N, sample_mode;
  const int32_t* ctx;
  int64_t ctx_stride;
  const int32_t* ctx_len;
  int32_t *tokens, *parents, *depth, *pos_ids;
  uint32_t* mask;
  int32_t *n_nodes, *match_n;
  int64_t* match_range;
  int32_t *node_count, *status;
  rest::BucketIndex idx;
  int nwords;   // bitmap words per depth
  int kcap;     // rows the block's shared memory holds, a multiple of 32
  // three-launch form of the batched path: the search launch sorts the contexts that matched
  // into two lists by candidate count, the two build launches take one list each
  int32_t* list;          // [2][B] context indices
  int32_t* list_count;    // [2]
  int B;
  int which;              // list of this build launch
  int light_rows;         // candidate counts up to this go to list 0
};

// Three-way comparison of the first n tokens of the suffix stored in slot `slot` with q.
// -1 / 0 / +1; a suffix that ends early is smaller.  An out-of-range suffix-array entry
// compares as smaller and raises `bad`.
template <typename SaT>
__device__ __forceinline__ int probe(const int32_t* __restrict__ T, const SaT* __restrict__ sa,
                                     int64_t n_tokens, int64_t slot, const int (&q)[16], int n,
                                     bool& bad) {
  int64_t p = (int64_t)__ldg(sa + slot);
  if (p < 0 || p >= n_tokens) { bad = true; return -1; }
  const int64_t rem = n_tokens - p;
  const int avail = rem < (int64_t)n ? (int)rem : n;     // tokens of the suffix that exist
  const int32_t* __restrict__ row = T + p;
  int tk[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) tk[k] = (k < avail) ? __ldg(row + k) : 0;
  int r = avail < n ? -1 : 0;                            // equal so far, but it ends early: smaller
#pragma unroll
  for (int k = 15; k >= 0; --k) {
    if (k < avail) {
      uint32_t a = (uint32_t)tk[k], b = (uint32_t)q[k];
      if (a != b) r = a < b ? -1 : 1;
    }
  }
  return r;
}

// First slot in [lo, hi) whose comparison is >= 0 (STRICT = false) or > 0 (STRICT = true);
// hi when there is none.  Warp-cooperative; all lanes return the same value.  `eq` reports
// whether the returned slot compared equal (in: whether slot `hi` is known to compare equal).
// `next_gt` (STRICT = false only): the first slot that compares greater, when the last round's
// probes happen to show it (the run of equal slots ends inside the last 32 probed slots, or runs
// up to a slot already known to be greater); -1 when it is not known.
//
// A = 32: every round all 32 lanes probe (fewest dependent rounds: the single-context path).
// A < 32: only the first WIDE rounds are 32 wide (a search over the whole array: their probe
// positions are the top of a fixed 33-ary tree, the same for every context, and stay in L2); the rounds
// below them, whose probes go to DRAM, use A lanes (A probes cut the interval into A + 1
// parts), which costs more dependent rounds but far fewer random DRAM reads per search.
template <typename SaT, bool STRICT, int A = 32, int WIDE = kWideRounds>
__device__ int64_t warp_first_true(const int32_t* __restrict__ T, const SaT* __restrict__ sa,
                                   int64_t n_tokens, int64_t lo, int64_t hi, const int (&q)[16],
                                   int n, int lane, bool& eq, bool& bad, int64_t* next_gt = nullptr) {
  // floor(2^64 / (A + 1))
  constexpr unsigned long long kInv = A == 32 ? 0x07C1F07C1F07C1F0ull : ~0ull / (unsigned long long)(A + 1);
  int round = 0;
  while (hi - lo > A) {
    int64_t size = hi - lo;
    const bool wide = A == 32 || (round < WIDE && size > 32);
    ++round;
    // P probes that cut the interval into P + 1 parts: floor((lane + 1) * size * floor(2^64 /
    // (P + 1)) / 2^64) is at most (lane + 1) * size / (P + 1), non-decreasing in the lane, and
    // below size; which slots are probed does not change the answer, only how fast the
    // interval shrinks
    const int last = wide ? 31 : A - 1;
    int64_t pos = lo + (int64_t)__umul64hi((unsigned long long)(lane + 1) * (unsigned long long)size,
                                           wide ? 0x07C1F07C1F07C1F0ull : kInv);
    int c = 1;
    if (lane <= last) c = probe<SaT>(T, sa, n_tokens, pos, q, n, bad);
    bool t = STRICT ? (c > 0) : (c >= 0);
    unsigned b = __ballot_sync(kFull, t && lane <= last);
    if (b == 0) {
      lo = __shfl_sync(kFull, pos, last) + 1;
    } else {
      int f = __ffs(b) - 1;
      int64_t pf = __shfl_sync(kFull, pos, f);
      int cf = __shfl_sync(kFull, c, f);
      int64_t pprev = __shfl_sync(kFull, pos, f > 0 ? f - 1 : 0);
      hi = pf;
      eq = (cf == 0);
      if (f > 0) lo = pprev + 1;
    }
  }
  int64_t pos = lo + lane;
  int c = -1;
  if (pos < hi) c = probe<SaT>(T, sa, n_tokens, pos, q, n, bad);
  bool t = (pos < hi) && (STRICT ? (c > 0) : (c >= 0));
  unsigned b = __ballot_sync(kFull, t);
  if (!STRICT && next_gt) {
    // slot hi compares greater unless `eq` says it is equal (hi = end of the array counts as greater)
    const unsigned gt = __ballot_sync(kFull, (pos < hi) && c > 0);
    *next_gt = gt ? lo + (__ffs(gt) - 1) : (eq ? (int64_t)-1 : hi);
  }
  if (b != 0) {
    int f = __ffs(b) - 1;
    int cf = __shfl_sync(kFull, c, f);
    eq = (cf == 0);
    return lo + f;
  }
  return hi;
}

// Suffix-array slot of candidate j.
__device__ __forceinline__ int64_t sample_slot(int64_t lo, int64_t cnt, int K, int mode, int j) {
  if (cnt <= (int64_t)K || mode == REST_SAMPLE_FIRST_K) return lo + j;
  return lo + (int64_t)(((unsigned long long)j * (unsigned long long)cnt) / (unsigned long long)K);
}

// Smallest set bit strictly after position j (the bitmap carries a sentinel past the rows).
// jump[w] holds the position of the first set bit in the words after w, so a run that spans
// many words costs one more load, not one per word.
__device__ __forceinline__ int next_set(const uint32_t* __restrict__ row,
                                        const uint16_t* __restrict__ jump, int j) {
  const int w = j >> 5;
  const uint32_t bits = row[w] & ~((2u << (j & 31)) - 1u);
  return bits ? (w << 5) + __ffs(bits) - 1 : (int)jump[w];
}

// Largest set bit at or before position j (bit 0 is always set).
__device__ __forceinline__ int prev_set(const uint32_t* __restrict__ row, int j) {
  int w = j >> 5;
  uint32_t bits = row[w] & ((2u << (j & 31)) - 1u);
  while (bits == 0 && w > 0) bits = row[--w];
  return (w << 5) + 31 - __clz(bits | 1u);
}

// Executed by one warp.  hist[0..nbins) holds counts; total >= need >= 1.  Finds the largest
// bin b with sum(hist[k], k > b) < need; returns b and that sum.
__device__ void warp_threshold_desc(const uint32_t* hist, int nbins, uint32_t need, int lane,
                                    int* out_bin, uint32_t* out_above) {
  int per = (nbins + 31) / 32;
  int top = nbins - 1 - lane * per;
  int bot = max(0, top - per + 1);
  uint32_t s = 0;
  for (int b = top; b >= bot && b >= 0; --b) s += hist[b];
  uint32_t incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t v = __shfl_up_sync(kFull, incl, o);
    if (lane >= o) incl += v;
  }
  uint32_t excl = incl - s;
  if (excl < need && need <= incl) {
    uint32_t acc = excl;
    for (int b = top; b >= bot; --b) {
      uint32_t h = hist[b];
      if (acc + h >= need) { *out_bin = b; *out_above = acc; break; }
      acc += h;
    }
  }
}

struct Smem {
  int q[16];
  long long lb[17], ub[17];
  uint32_t e1[kMaxM + 1];      // nodes of weight 1 per depth
  int e1diff[kMaxM + 2];       // the same as a difference array over depths, before the prefix sum
  uint32_t heavy_total;        // nodes of weight >= 2
  int err;
  int bin_hi;
  uint32_t above_hi;
  int bin_lo;
  uint32_t above_lo;
  uint32_t nsel;
  uint32_t warp_cnt[32];
  uint32_t sel[kMaxN];         // depth << 16 | row
  uint32_t selcnt[kMaxN];
  uint32_t sorted[kMaxN];
  uint32_t sortedcnt[kMaxN];
  int par[kMaxN];
  uint32_t hist_hi[kHistHi];
  uint32_t hist_lo[kHistLo];
};

// TP = false: the single-context path, tuned for the fewest dependent reads.  TP = true: the
// batched path, for calls with more contexts than the GPU holds at once; the same results by
// fewer random DRAM reads per context (see phase 1).
// PART: kWhole = search and build in one launch; kSearch = phase 1 only (writes match_n and
// match_range, the defaults of every output slot, and the context's index into one of two
// lists); kBuild = phases 2-4 for the contexts of one list.
enum { kWhole = 0, kSearch = 1, kBuild = 2 };
template <typename SaT, bool TP, int NT, int PART>
__global__ void __launch_bounds__(NT, 1024 / NT)
rest_draft_kernel(DraftArgs a) {
  constexpr int NW = NT / 32;
  static_assert(NT % 32 == 0 && NT >= 64, "whole warps; at least kMaxM + 2 threads");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem& s = *reinterpret_cast<Smem*>(smem_raw);
  uint16_t* lenlcp = reinterpret_cast<uint16_t*>(smem_raw + sizeof(Smem));          // [kcap]
  uint32_t* bm = reinterpret_cast<uint32_t*>(smem_raw + sizeof(Smem) + 2 * a.kcap); // [m][nwords]
  uint16_t* jump = reinterpret_cast<uint16_t*>(bm + a.m * a.nwords);                // [m][nwords]

  if constexpr (PART == kBuild) {
    if ((int)blockIdx.x >= a.list_count[a.which]) return;
  }
  const int b = PART == kBuild ? a.list[(int64_t)a.which * a.B + blockIdx.x] : (int)blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = a.N, m = a.m, Wm = (N + 31) >> 5;
  // a kernel launched behind this one with programmatic stream serialisation may begin its
  // set-up now (it still waits for this grid to complete before it reads anything)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int32_t* __restrict__ T = a.T;
  const SaT* __restrict__ sa = static_cast<const SaT*>(a.sa);
  const int64_t n_tokens = a.n_tokens;
  const int clen = a.ctx_len[b];
  const int32_t* ctx = a.ctx + (int64_t)b * a.ctx_stride;

  // Unused-slot defaults; thread i owns slots i, i + NT, ... for the whole kernel (a build
  // launch finds them written by the search launch).
  if constexpr (PART != kBuild)
  for (int i = tid; i < N; i += NT) {
    int64_t o = (int64_t)b * N + i;
    a.tokens[o] = -1; a.parents[o] = -1; a.depth[o] = 0; a.pos_ids[o] = clen;
    for (int w = 0; w < Wm; ++w) a.mask[o * Wm + w] = (w == (i >> 5)) ? (1u << (i & 31)) : 0u;
    if (a.node_count) a.node_count[o] = 0;
  }
  const int nq = min(a.n_max, max(clen, 0));   // context tokens that can take part
  if (tid == 0) { s.err = 0; s.heavy_total = 0; s.nsel = 0; }
  if (tid < 17) { s.lb[tid] = 0; s.ub[tid] = 0; }
  if (tid <= kMaxM) s.e1[tid] = 0;
  if (tid <= kMaxM + 1) s.e1diff[tid] = 0;
  if constexpr (PART != kSearch) {
    for (int i = tid; i < kHistHi; i += NT) s.hist_hi[i] = 0;
    for (int i = tid; i < kHistLo; i += NT) s.hist_lo[i] = 0;
  }
  __syncthreads();
  int n_win = 0;
  if constexpr (PART == kBuild) {
    n_win = a.match_n[b];
    if (tid == 0) { s.lb[n_win] = a.match_range[2 * b]; s.ub[n_win] = a.match_range[2 * b + 1]; }
    __syncthreads();
  } else {
  if (tid < nq) {
    int t = ctx[clen - nq + tid];
    s.q[tid] = t;
    if (t < 0 || (uint32_t)t >= a.vocab) atomicOr(&s.err, REST_CTX_BAD_TOKEN);
  }
  __syncthreads();
  if (s.err != 0 || nq < a.n_min) {
    if (tid == 0) {
      a.status[b] = s.err; a.n_nodes[b] = 0; a.match_n[b] = 0;
      a.match_range[2 * b] = 0; a.match_range[2 * b + 1] = 0;
    }
    return;
  }

  // ---- phase 1: search --------------------------------------------------------------
  // 1a: lower bound of every suffix length, one warp each.  ub = -1 marks "matches, end of the
  // run not known yet".
  constexpr int kArity = TP ? kTpArity : 32;
  auto lower_bound_of = [&](int n) {     // executed by one whole warp
    int q[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) q[k] = (k < n) ? s.q[nq - n + k] : 0;
    bool bad = false, eq = false;
    int64_t next_gt = -1;
    int64_t lb = warp_first_true<SaT, false, kArity>(T, sa, n_tokens, 0, n_tokens, q, n, lane, eq, bad, &next_gt);
    if (__any_sync(kFull, bad) && lane == 0) atomicOr(&s.err, REST_CTX_BAD_DATASTORE);
    if (lane == 0) { s.lb[n] = lb; s.ub[n] = (eq && lb < n_tokens) ? next_gt : lb; }
  };
  if constexpr (!TP || !kTpStaged) {
    for (int n = a.n_min + warp; n <= nq; n += NW) lower_bound_of(n);   // one length per warp when NW = 16
  } else {
    // If the suffix of length n occurs in the datastore, so does the one of length n - 1 (the
    // same occurrence, one token later): the lengths that match are n_min ... n* without a
    // gap.  Two steps of three or four searches find n* among up to 16 lengths: every fourth length
    // first, then the three lengths above the longest of those that matched.  Lengths never
    // searched keep lb = ub = 0, "no match", which is what they are.
    const int nlen = nq - a.n_min + 1;
    if (warp < 4) {
      const int i = 3 + 4 * warp;
      if (i < nlen) lower_bound_of(a.n_min + i);
    }
    __syncthreads();
    int first = 0;
    for (int w = 3; w >= 0; --w) {
      const int i = 3 + 4 * w;
      if (i < nlen && s.ub[a.n_min + i] != s.lb[a.n_min + i]) { first = i + 1; break; }
    }
    if (warp < 3) {
      const int i = first + warp;
      if (i < nlen) lower_bound_of(a.n_min + i);
    }
  }
  __syncthreads();
  for (int n = nq; n >= a.n_min; --n)
    if (s.ub[n] != s.lb[n]) { n_win = n; break; }
  // 1b: only the winning length needs its upper bound, and only if the last round of its lower
  // bound did not already show where the run ends (shorter lengths match far more slots and
  // would need the most rounds: they are never looked at again)
  if (n_win != 0 && s.ub[n_win] < 0) {       // block-uniform
    if (warp == (n_win - a.n_min) % NW) {
      const int n = n_win;
      int q[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) q[k] = (k < n) ? s.q[nq - n + k] : 0;
      bool bad = false;
      const int64_t lb = s.lb[n];
      // gallop: slot lb + 2^e for e = 0 ... 31, all at once or kArity exponents per round; f =
      // the first exponent whose slot compares greater or lies past the end (-1: none)
      int f = -1;
      for (int g = 0; g < 32 / kArity; ++g) {
        bool t = false;
        if (lane < kArity) {
          const int64_t pos = lb + ((int64_t)1 << (g * kArity + lane));
          t = true;
          if (pos < n_tokens) t = probe<SaT>(T, sa, n_tokens, pos, q, n, bad) > 0;
        }
        const unsigned bal = __ballot_sync(kFull, t);
        if (bal != 0) { f = g * kArity + __ffs(bal) - 1; break; }
      }
      int64_t lo2, hi2 = n_tokens;
      bool eq2 = false;
      if (f < 0) {
        lo2 = lb + ((int64_t)1 << 31) + 1;
      } else {
        int64_t pf = lb + ((int64_t)1 << f);
        hi2 = pf < n_tokens ? pf : n_tokens;
        lo2 = f > 0 ? lb + ((int64_t)1 << (f - 1)) + 1 : lb + 1;
      }
      if (lo2 > hi2) lo2 = hi2;
      const int64_t ub = warp_first_true<SaT, true, kArity, 0>(T, sa, n_tokens, lo2, hi2, q, n, lane, eq2, bad);
      if (__any_sync(kFull, bad) && lane == 0) atomicOr(&s.err, REST_CTX_BAD_DATASTORE);
      if (lane == 0) s.ub[n] = ub;
    }
    __syncthreads();
  }
  if (s.err != 0 || n_win == 0) {
    if (tid == 0) {
      a.status[b] = s.err; a.n_nodes[b] = 0; a.match_n[b] = 0;
      a.match_range[2 * b] = 0; a.match_range[2 * b + 1] = 0;
    }
    return;
  }
  }  // PART != kBuild
  const int64_t lo = s.lb[n_win], hi = s.ub[n_win];
  const int64_t cnt = hi - lo;
  if constexpr (PART == kSearch) {
    // hand the context to the build launch that fits its candidate count
    if (tid == 0) {
      a.status[b] = 0; a.n_nodes[b] = 0; a.match_n[b] = n_win;
      a.match_range[2 * b] = lo; a.match_range[2 * b + 1] = hi;
      const int heavy = (cnt < (int64_t)a.K ? cnt : (int64_t)a.K) > (int64_t)a.light_rows;
      const int at = atomicAdd(a.list_count + heavy, 1);
      a.list[(int64_t)heavy * a.B + at] = b;
    }
    return;
  }
  const int Kp = (int)(cnt < (int64_t)a.K ? cnt : (int64_t)a.K);
  const int nwords = a.nwords;
  const int niter = (Kp + NT - 1) / NT;

  // ---- phase 2: gather rows, common-prefix lengths, node-start bitmaps --------------------
  // the suffix-array entry of the next iteration's row is fetched one iteration ahead, so
  // that the two dependent reads (entry, then tokens) of consecutive iterations overlap
  // (lane 0 also needs the row before its own, which another warp holds: it fetches that
  // entry ahead as well and reads both rows' tokens side by side)
  int64_t p_next = 0, pp_next = 0;
  if (tid < Kp) p_next = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, tid));
  if (lane == 0 && tid > 0 && tid <= Kp)
    pp_next = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, tid - 1));
  for (int it = 0; it < niter; ++it) {
    const int jbase = it * NT + warp * 32;
    const int j = jbase + lane;
    int64_t p = p_next;
    const int64_t pp = pp_next;
    if (j + NT < Kp) p_next = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, j + NT));
    if (lane == 0 && j + NT <= Kp)
      pp_next = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, j + NT - 1));
    if (jbase >= Kp) continue;   // warp-uniform
    const bool valid = j < Kp;
    int row[kMaxM], prev[kMaxM];
    int len = 0, plen = 0;
    bool bad = false;
    if (valid) {
      if (p < 0 || p >= n_tokens) { bad = true; p = 0; }
      int64_t base = p + n_win;
      int64_t rem = n_tokens - base;
      len = bad ? 0 : (int)(rem < 0 ? 0 : (rem > m ? m : rem));
#pragma unroll
      for (int d = 0; d < kMaxM; ++d) row[d] = (d < len) ? __ldg(T + base + d) : 0;
    } else {
#pragma unroll
      for (int d = 0; d < kMaxM; ++d) row[d] = 0;
    }
#pragma unroll
    for (int d = 0; d < kMaxM; ++d) prev[d] = __shfl_up_sync(kFull, row[d], 1);
    plen = __shfl_up_sync(kFull, len, 1);
    if (lane == 0 && j > 0) {   // previous row belongs to another warp: fetch it again
      int64_t p = pp;
      if (p < 0 || p >= n_tokens) { bad = true; p = 0; }
      int64_t base = p + n_win;
      int64_t rem = n_tokens - base;
      plen = bad ? 0 : (int)(rem < 0 ? 0 : (rem > m ? m : rem));
#pragma unroll
      for (int d = 0; d < kMaxM; ++d) prev[d] = (d < plen) ? __ldg(T + base + d) : 0;
    }
    int lcp = 0;
    if (valid && j > 0) {
      const int lim = min(len, plen);
      bool run = true;
      bool ordered = plen <= len;   // decides when one row is a prefix of the other
#pragma unroll
      for (int d = 0; d < kMaxM; ++d) {
        if (run && d < lim) {
          if (row[d] == prev[d]) {
            lcp = d + 1;
          } else {
            run = false;
            ordered = (uint32_t)prev[d] < (uint32_t)row[d];
          }
        }
      }
      if (!ordered) bad = true;
    }
    if (valid) lenlcp[j] = (uint16_t)(lcp | (len << 8));
    uint32_t myword = 0;
#pragma unroll
    for (int d = 1; d <= kMaxM; ++d) {
      if (d <= m) {
        uint32_t w = __ballot_sync(kFull, !valid || lcp < d);
        if (lane == d - 1) myword = w;
      }
    }
    if (lane < m) bm[lane * nwords + (jbase >> 5)] = myword;
    if (__any_sync(kFull, bad) && lane == 0) atomicOr(&s.err, REST_CTX_BAD_DATASTORE);
  }
  if (tid < m) bm[tid * nwords + ((Kp + 31) >> 5)] = kFull;   // sentinel past the last row
  __syncthreads();
  if (s.err != 0) {
    if (tid == 0) {
      a.status[b] = s.err; a.n_nodes[b] = 0; a.match_n[b] = 0;
      a.match_range[2 * b] = 0; a.match_range[2 * b + 1] = 0;
    }
    return;
  }

  // jump table: for every depth (a warp each) a suffix scan over the bitmap words, last chunk
  // of 32 words first: jump[w] = position of the first set bit in any word after w
  for (int dd = warp; dd < m; dd += NW) {
    const uint32_t* row = bm + dd * nwords;
    uint16_t* jrow = jump + dd * nwords;
    const int last = (Kp + 31) >> 5;              // the sentinel word
    int carry = 0x7FFFFFFF;
    for (int c = last >> 5; c >= 0; --c) {
      const int wi = c * 32 + lane;
      const uint32_t bits = wi <= last ? row[wi] : 0u;
      int v = bits ? (wi << 5) + __ffs(bits) - 1 : 0x7FFFFFFF;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {          // inclusive suffix minimum over the lanes
        const int u = __shfl_down_sync(kFull, v, o);
        if (lane + o < 32) v = min(v, u);
      }
      v = min(v, carry);
      const int after = __shfl_down_sync(kFull, v, 1);
      if (wi <= last) jrow[wi] = (uint16_t)min(lane < 31 ? after : carry, 0xFFFF);
      carry = __shfl_sync(kFull, v, 0);
    }
  }
  __syncthreads();

  // ---- phase 3a: histogram of (weight, depth) over all Trie nodes --------------------------
  // key = weight << 5 | (16 - depth): larger key = better node.
  for (int it = 0; it < niter; ++it) {
    const int jbase = it * NT + warp * 32;
    if (jbase >= Kp) continue;
    const int j = jbase + lane;
    const bool valid = j < Kp;
    const int ll = valid ? lenlcp[j] : 0;
    const int lcp = ll & 0xFF, len = ll >> 8;
    // Weights along a row never grow with depth: walk down from the first depth at which the
    // row starts a node until the weight drops to 1; every deeper node of the row weighs 1.
    uint32_t nheavy = 0;
    int d1 = len + 1;                      // first depth of weight 1 (len + 1: none)
    if (valid) {
      for (int d = lcp + 1; d <= len; ++d) {
        const int c = next_set(bm + (d - 1) * nwords, jump + (d - 1) * nwords, j) - j;
        if (c < 2) { d1 = d; break; }
        atomicAdd(&s.hist_hi[((c << 5) | (16 - d)) >> 10], 1u);
        ++nheavy;
      }
    }
    // weight-1 nodes per depth: d1 <= d <= len, counted as starts minus ends per warp
    for (int d = 1; d <= m + 1; ++d) {
      const uint32_t st = __ballot_sync(kFull, valid && d1 == d && d1 <= len);
      const uint32_t en = __ballot_sync(kFull, valid && d1 <= len && len + 1 == d);
      if (lane == 0 && (st | en)) atomicAdd(&s.e1diff[d], __popc(st) - __popc(en));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nheavy += __shfl_xor_sync(kFull, nheavy, o);
    if (lane == 0 && nheavy) atomicAdd(&s.heavy_total, nheavy);
  }
  __syncthreads();

  if (tid == 0) {
    int run = 0;
    for (int d = 1; d <= m; ++d) { run += s.e1diff[d]; s.e1[d] = (uint32_t)run; }
  }
  __syncthreads();

  // ---- phase 3b: threshold key t*, number of ties wanted ------------------------------------
  uint32_t tstar;      // nodes with key > tstar are kept
  uint32_t r_tie;      // plus the first r_tie nodes (by row) with key == tstar
  const uint32_t heavy_total = s.heavy_total;
  if (heavy_total >= (uint32_t)N) {
    if (warp == 0) warp_threshold_desc(s.hist_hi, kHistHi, (uint32_t)N, lane, &s.bin_hi, &s.above_hi);
    __syncthreads();
    const int bin_hi = s.bin_hi;
    for (int it = 0; it < niter; ++it) {
      const int jbase = it * NT + warp * 32;
      if (jbase >= Kp) continue;
      const int j = jbase + lane;
      if (j >= Kp) continue;
      const int ll = lenlcp[j];
      const int lcp = ll & 0xFF, len = ll >> 8;
      for (int d = lcp + 1; d <= len; ++d) {
        int c = next_set(bm + (d - 1) * nwords, jump + (d - 1) * nwords, j) - j;
        if (c < 2) break;   // weights do not grow with depth
        uint32_t key = ((uint32_t)c << 5) | (uint32_t)(16 - d);
        if ((int)(key >> 10) == bin_hi) atomicAdd(&s.hist_lo[key & 1023u], 1u);
      }
    }
    __syncthreads();
    if (warp == 0)
      warp_threshold_desc(s.hist_lo, kHistLo, (uint32_t)N - s.above_hi, lane, &s.bin_lo, &s.above_lo);
    __syncthreads();
    tstar = ((uint32_t)bin_hi << 10) | (uint32_t)s.bin_lo;
    r_tie = (uint32_t)N - s.above_hi - s.above_lo;
  } else {
    // every node of weight >= 2 is kept; weight-1 nodes fill up by depth, then by row
    uint32_t need = (uint32_t)N - heavy_total, cum = 0;
    tstar = 0; r_tie = 0;
    for (int d = 1; d <= m; ++d) {
      uint32_t e = s.e1[d];
      if (cum + e >= need) { tstar = (1u << 5) | (uint32_t)(16 - d); r_tie = need - cum; break; }
      cum += e;
    }
  }
  const int d_tie = 16 - (int)(tstar & 31u);
  const int c_tie = (int)(tstar >> 5);

  // ---- phase 3c: collect the kept nodes -----------------------------------------------------
  uint32_t tie_base = 0;
  for (int it = 0; it < niter; ++it) {
    const int j = it * NT + tid;
    const bool valid = j < Kp;
    bool tie = false;
    if (valid) {
      const int ll = lenlcp[j];
      const int lcp = ll & 0xFF, len = ll >> 8;
      for (int d = lcp + 1; d <= len; ++d) {
        int c = next_set(bm + (d - 1) * nwords, jump + (d - 1) * nwords, j) - j;
        uint32_t key = ((uint32_t)c << 5) | (uint32_t)(16 - d);
        if (key > tstar) {
          uint32_t slot = atomicAdd(&s.nsel, 1u);
          if (slot < (uint32_t)N) { s.sel[slot] = ((uint32_t)d << 16) | (uint32_t)j; s.selcnt[slot] = c; }
        } else {
          tie = key == tstar;
          break;                           // keys only fall with depth along a row
        }
      }
    }
    if (r_tie > 0) {   // block-uniform
      uint32_t bal = __ballot_sync(kFull, tie);
      if (lane == 0) s.warp_cnt[warp] = __popc(bal);
      __syncthreads();
      uint32_t before = tie_base, total = 0;
      for (int w = 0; w < NW; ++w) {
        uint32_t c = s.warp_cnt[w];
        if (w < warp) before += c;
        total += c;
      }
      uint32_t rank = before + __popc(bal & ((1u << lane) - 1u));
      if (tie && rank < r_tie) {
        uint32_t slot = atomicAdd(&s.nsel, 1u);
        if (slot < (uint32_t)N) { s.sel[slot] = ((uint32_t)d_tie << 16) | (uint32_t)j; s.selcnt[slot] = c_tie; }
      }
      tie_base += total;
      __syncthreads();
    }
  }
  __syncthreads();
  const int nn = (int)min(s.nsel, (uint32_t)N);
  if (s.nsel > (uint32_t)N && tid == 0) atomicOr(&s.err, REST_CTX_INTERNAL);

  // ---- phase 4: breadth-first order, parents, masks, tokens ---------------------------------
  for (int i = tid; i < nn; i += NT) {
    const uint32_t me = s.sel[i];
    int rank = 0;
    for (int k = 0; k < nn; ++k) rank += (s.sel[k] < me);
    s.sorted[rank] = me;
    s.sortedcnt[rank] = s.selcnt[i];
  }
  __syncthreads();
  for (int i = tid; i < nn; i += NT) {
    const uint32_t me = s.sorted[i];
    const int d = (int)(me >> 16), j = (int)(me & 0xFFFFu);
    int par = -1;
    if (d > 1) {
      const int jp = prev_set(bm + (d - 2) * nwords, j);
      const uint32_t pkey = ((uint32_t)(d - 1) << 16) | (uint32_t)jp;
      int l = 0, r = nn - 1;
      par = -2;
      while (l <= r) {
        int mid = (l + r) >> 1;
        uint32_t v = s.sorted[mid];
        if (v == pkey) { par = mid; break; }
        if (v < pkey) l = mid + 1; else r = mid - 1;
      }
      if (par < 0) { atomicOr(&s.err, REST_CTX_INTERNAL); par = -1; }
    }
    s.par[i] = par;
    int64_t p = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, j));
    int64_t o = (int64_t)b * N + i;
    a.tokens[o] = __ldg(T + p + n_win + d - 1);
    a.parents[o] = par;
    a.depth[o] = d;
    a.pos_ids[o] = clen + d - 1;
    if (a.node_count) a.node_count[o] = (int32_t)s.sortedcnt[i];
  }
  __syncthreads();
  for (int i = tid; i < nn; i += NT) {
    uint32_t bits[(kMaxN + 31) / 32];
#pragma unroll
    for (int w = 0; w < (kMaxN + 31) / 32; ++w) bits[w] = 0;
    int k = i;
    for (int step = 0; step <= kMaxM && k >= 0; ++step) {
#pragma unroll
      for (int w = 0; w < (kMaxN + 31) / 32; ++w)
        if (w == (k >> 5)) bits[w] |= 1u << (k & 31);
      k = s.par[k];
    }
    int64_t o = ((int64_t)b * N + i) * Wm;
#pragma unroll
    for (int w = 0; w < (kMaxN + 31) / 32; ++w)
      if (w < Wm) a.mask[o + w] = bits[w];
  }
  __syncthreads();
  if (s.err != 0) {
    // an inconsistency met while the tree was being written: the caller gets the empty tree
    // that every other reported problem gives, not a half-built one
    for (int i = tid; i < N; i += NT) {
      int64_t o = (int64_t)b * N + i;
      a.tokens[o] = -1; a.parents[o] = -1; a.depth[o] = 0; a.pos_ids[o] = clen;
      for (int w = 0; w < Wm; ++w) a.mask[o * Wm + w] = (w == (i >> 5)) ? (1u << (i & 31)) : 0u;
      if (a.node_count) a.node_count[o] = 0;
    }
  }
  if (tid == 0) {
    const bool ok = s.err == 0;
    a.status[b] = s.err;
    a.n_nodes[b] = ok ? nn : 0;
    a.match_n[b] = ok ? n_win : 0;
    a.match_range[2 * b] = ok ? lo : 0;
    a.match_range[2 * b + 1] = ok ? hi : 0;
  }
}

size_t draft_smem_bytes(int K, int m, int* kcap_out, int* nwords_out) {
  int kcap = (K + 31) / 32 * 32;
  int nwords = kcap / 32 + 1;
  if (kcap_out) *kcap_out = kcap;
  if (nwords_out) *nwords_out = nwords;
  size_t bytes = sizeof(Smem) + 2 * (size_t)kcap + (4 + 2) * (size_t)m * nwords;
  return (bytes + 15) / 16 * 16;
}

}  // namespace

// Whether a call of B contexts takes the batched path (search = the REST_SEARCH_* bits;
// with_scratch: the caller gives the scratch of the three-launch form).
static rest_status wants_batched(int search, int B, bool with_scratch, bool* batched) {
  *batched = search == REST_SEARCH_BATCHED;
  if (search == REST_SEARCH_AUTO) {
    // Below a few contexts per SM a call lasts as long as its slowest contexts and the shortest
    // dependent chain wins.  Measured crossover on 148 SMs: between 512 and 1024 contexts for the
    // three-launch form, between 1024 and 4096 for the one-launch form.
    const int sms = rest::sm_count();
    if (sms <= 0) return rest::note_cuda_error(cudaErrorNoDevice, "sm_count");
    *batched = B >= (with_scratch ? 5 : 16) * sms;
  }
  return REST_OK;
}

static size_t split_workspace_bytes(int B) { return (2 * (size_t)B + 16) * sizeof(int32_t); }

extern "C" size_t rest_draft_workspace_bytes(const rest_draft_params* prm, int32_t B) {
  if (!prm || B <= 0) return 0;
  bool batched = false;
  if (wants_batched(prm->search_path, B, true, &batched) != REST_OK || !batched) return 0;
  return split_workspace_bytes(B);
}

extern "C" rest_status rest_draft(const rest_datastore* ds, const rest_draft_params* prm,
                                  const int32_t* d_ctx, int64_t ctx_stride,
                                  const int32_t* d_ctx_len, int32_t B, int32_t* d_tokens,
                                  int32_t* d_parents, int32_t* d_depth, int32_t* d_pos_ids,
                                  uint32_t* d_mask, int32_t* d_n_nodes, int32_t* d_match_n,
                                  int64_t* d_match_range, int32_t* d_node_count,
                                  int32_t* d_status, void* d_ws, size_t ws_bytes,
                                  void* stream) {
  if (!ds || !prm || B < 0) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_ctx || !d_ctx_len || !d_tokens || !d_parents || !d_depth || !d_pos_ids || !d_mask ||
      !d_n_nodes || !d_match_n || !d_match_range || !d_status || ctx_stride < 0)
    return REST_INVALID_ARG;
  if (prm->n_min < 1 || prm->n_max < prm->n_min || prm->K < 1 || prm->m < 1 || prm->N < 1)
    return REST_INVALID_ARG;
  const int sample_mode = prm->sample_mode;
  const int search = prm->search_path;
  if (sample_mode != REST_SAMPLE_STRIDED && sample_mode != REST_SAMPLE_FIRST_K)
    return REST_INVALID_ARG;
  if (search != REST_SEARCH_AUTO && search != REST_SEARCH_SINGLE && search != REST_SEARCH_BATCHED)
    return REST_INVALID_ARG;
  if (prm->n_max > REST_MAX_SUFFIX || prm->m > REST_MAX_M || prm->N > REST_MAX_N ||
      prm->K > REST_MAX_K || prm->n_max - prm->n_min + 1 > kWarps)
    return REST_UNSUPPORTED;

  DraftArgs a;
  a.T = ds->v.tokens; a.sa = ds->v.sa; a.n_tokens = ds->v.n_tokens; a.vocab = ds->v.vocab;
  a.n_max = prm->n_max; a.n_min = prm->n_min; a.K = prm->K; a.m = prm->m; a.N = prm->N;
  a.sample_mode = sample_mode;
  a.ctx = d_ctx; a.ctx_stride = ctx_stride; a.ctx_len = d_ctx_len;
  a.tokens = d_tokens; a.parents = d_parents; a.depth = d_depth; a.pos_ids = d_pos_ids;
  a.mask = d_mask; a.n_nodes = d_n_nodes; a.match_n = d_match_n; a.match_range = d_match_range;
  a.node_count = d_node_count; a.status = d_status;
  size_t smem = draft_smem_bytes(prm->K, prm->m, &a.kcap, &a.nwords);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool with_scratch = d_ws && ws_bytes >= split_workspace_bytes(B);
  bool batched = false;
  if (rest_status rc = wants_batched(search, B, with_scratch, &batched); rc != REST_OK) return rc;
  const bool narrow = ds->v.sa_bytes == 4;
  a.list = nullptr; a.list_count = nullptr; a.B = B; a.which = 0; a.light_rows = 0;
  auto launch = [&](auto kern, int slot, int threads, int blocks, size_t bytes) -> rest_status {
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(kern),
                                            rest::kSmemSlotDraft + slot + (narrow ? 0 : 1), bytes));
    kern<<<blocks, threads, bytes, st>>>(a);
    rest::count_launch();
    REST_CUDA_TRY(cudaGetLastError());
    return REST_OK;
  };
  const bool big = smem > kBigSmemBytes;
  if (!batched) {
    // a call with at most one context per SM lasts as long as its slowest context: give each
    // context the whole SM (not the single context: its typical candidate list is short and
    // the larger block only adds barrier time)
    const int sms = rest::sm_count();
    if (big || (B > 1 && B <= sms))
      return narrow ? launch(rest_draft_kernel<int32_t, false, kBigThreads, kWhole>, 10, kBigThreads, B, smem)
                    : launch(rest_draft_kernel<int64_t, false, kBigThreads, kWhole>, 10, kBigThreads, B, smem);
    return narrow ? launch(rest_draft_kernel<int32_t, false, kThreads, kWhole>, 0, kThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, false, kThreads, kWhole>, 0, kThreads, B, smem);
  }
  if (!with_scratch) {
    // no scratch for the context lists: search and build in one launch
    return narrow ? launch(rest_draft_kernel<int32_t, true, kTpThreads, kWhole>, 2, kTpThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, true, kTpThreads, kWhole>, 2, kTpThreads, B, smem);
  }
  // Three launches: the search with a small block per context; then the contexts that matched,
  // those with few candidates on small blocks (many per SM) and the others on large ones.  A
  // build launch has one block per context of the call; the blocks beyond its list leave at once.
  a.list_count = static_cast<int32_t*>(d_ws);
  a.list = a.list_count + 16;
  a.light_rows = prm->K < kLightRows ? prm->K : kLightRows;
  REST_CUDA_TRY(cudaMemsetAsync(a.list_count, 0, 2 * sizeof(int32_t), st));
  rest_status rc = narrow ? launch(rest_draft_kernel<int32_t, true, kSearchThreads, kSearch>, 4, kSearchThreads, B, sizeof(Smem))
                          : launch(rest_draft_kernel<int64_t, true, kSearchThreads, kSearch>, 4, kSearchThreads, B, sizeof(Smem));
  if (rc != REST_OK) return rc;
  const int kcap_all = a.kcap, nwords_all = a.nwords;
  const size_t smem_light = draft_smem_bytes(a.light_rows, prm->m, &a.kcap, &a.nwords);
  a.which = 0;
  rc = narrow ? launch(rest_draft_kernel<int32_t, true, kLightThreads, kBuild>, 6, kLightThreads, B, smem_light)
              : launch(rest_draft_kernel<int64_t, true, kLightThreads, kBuild>, 6, kLightThreads, B, smem_light);
  if (rc != REST_OK) return rc;
  if (prm->K > a.light_rows) {
    a.kcap = kcap_all; a.nwords = nwords_all; a.which = 1;
    if (big)
      rc = narrow ? launch(rest_draft_kernel<int32_t, true, kBigThreads, kBuild>, 12, kBigThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, true, kBigThreads, kBuild>, 12, kBigThreads, B, smem);
    else
      rc = narrow ? launch(rest_draft_kernel<int32_t, true, kThreads, kBuild>, 8, kThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, true, kThreads, kBuild>, 8, kThreads, B, smem);
  }
  return rc;
}
