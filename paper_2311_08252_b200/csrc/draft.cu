// rest_draft: Algorithm 1 (longest-suffix retrieval over a suffix array), Algorithm 2
// (Trie weights and the c heaviest nodes) and the breadth-first pseudo sequence with its
// ancestor mask (Sec. 3.2), one thread block per context, everything in one launch (three
// for calls with thousands of contexts).
//
// Phases inside the block:
//   1 search   a warp per suffix length.  The datastore's n-gram index (when it has one) gives
//              the suffix-array range of the query's first two to four tokens in one read - the
//              answer itself for a short frequent suffix - and a 32-ary lower bound inside it
//              (every lane probes one slot per round, a ballot narrows the interval) finds the
//              first match.  Its probes also bracket the end of the run; only the longest
//              length that matched searches inside its bracket for the end.
//   2 gather   candidate rows in suffix-array order, which is also the lexicographic order of
//              the continuations.  A warp takes 32 rows (one bitmap word) at a time; a load
//              instruction fetches two rows, 16 columns each, and every token is compared with
//              the one above it where it sits.  Only the common-prefix length with the previous
//              row survives: for every depth d the bitmap "row j starts a new Trie node at
//              depth d" (lcp_j < d).  A context with thousands of rows shares them with blocks
//              that have nothing else to do (see ShareDesc).
//   3 select   weight of node (d, j) = distance to the next set bit of bitmap d.  All passes
//              run over (depth, bitmap word) pairs, not over rows: nodes of weight 1 to 4 are
//              read off the bit pattern of a word and counted with a popcount each, heavier
//              nodes are listed and weighed by a thread each.  The N largest by (weight desc,
//              depth asc, row asc) come from a two-level radix histogram over (weight, depth)
//              and a prefix sum over the words of the tie depth.
//   4 emit     rank the kept nodes by (depth, row), find parents by a predecessor search among
//              them, build ancestor masks, fetch the node tokens.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxM = REST_MAX_M;
constexpr int kMaxN = REST_MAX_N;
constexpr int kHistHi = 2080;   // first-level bins: weights below 1024 one by one, then 1024 + weight / 32
constexpr int kHistLo = 1024;
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kMaxTrunc = 32;                         // rows cut short by the end of the stream (at most m exist)
constexpr int kRowLoads = 17;                         // load instructions for a warp's 33 rows, two rows each
constexpr int kBigListCap = 4096;                     // nodes of weight >= 5 a block can list
constexpr int kPositionCacheRows = 1024;              // rows whose suffix position stays in shared memory for phase 4
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
constexpr size_t kBigRowsTimesM = 160000;   // K * m from which a context gets a 1024-thread block

struct DraftArgs {
  const int32_t* T;
  const void* sa;
  int64_t n_tokens;
  int64_t n_sa;
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
  int pcache_rows;   // rows whose suffix position is kept in shared memory
  int bigcap;        // nodes of weight >= 5 the block can list (an even number)
  // rows handed in by the caller as R sorted runs per context (rest_draft_from_runs): T then
  // points at the rows [B][R][Kr][m]
  const int32_t* row_len;     // [B][R][Kr]
  const int32_t* run_rows;    // [B][R]
  uint32_t* order;            // [B][kcap] scratch: merged order of the rows
  int R, Kr;
  // three-launch form of the batched path: the search launch sorts the contexts that matched
  // into two lists by candidate count, the two build launches take one list each
  int32_t* list;          // [2][B] context indices
  int32_t* list_count;    // [2]
  int B;
  int which;              // list of this build launch
  int light_rows;         // candidate counts up to this go to list 0
  // one-launch form with shared gathering (kWholeShare): see ShareDesc
  int32_t* sh_hdr = nullptr;        // counters, zeroed before the launch like sh_ready and sh_desc
  int32_t* sh_ready = nullptr;      // [B] 0: not offered, 1: chunks to claim, 2: all claimed
  struct ShareDesc* sh_desc = nullptr;   // [B]
  uint32_t* sh_trunc = nullptr;     // [B][kMaxTrunc]
  uint32_t* sh_bm = nullptr;        // [B][m][nwords]
  int share_rows = 0;         // a context with more candidates than this offers its gather to other blocks
};

// Shared gathering.  In a call with few contexts a call lasts as long as its slowest context, and
// what makes a context slow is a long candidate list, whose rows one block reads alone while the
// blocks of the other contexts have finished and other SMs never had a block.  So a context
// with many candidates publishes its matched range, and every warp that has nothing else to do
// - the warps of blocks whose own rows are read or whose context is finished, the warps of
// blocks launched as helpers only - takes bitmap words (32 rows each) off the END of its list:
// a block claims one word per warp with one atomic on the context's `back` counter, computes
// them into the scratch and counts them done.  The owner meanwhile works up from word 0 at its
// usual pace, looking at `back` before every word; when its warps have met the helpers it closes
// the counter, waits for the words that running warps still hold, reads the helpers' part of
// the bitmaps back and goes on alone.  A word may be computed twice where the two meet (the
// owner sees `back` one word late): both write the same bits, to different places.  Nothing
// depends on a helper being there: helpers that find nothing to do leave.
struct ShareDesc {
  long long lo, cnt;       // matched suffix-array range
  int Kp, n_win, nw;       // rows taken, matched length, bitmap words that hold rows
  int back;                // helpers hold the words from here to nw (atomic; the owner works up from word 0)
  int floor;               // words below this one are the owner's, whatever happens (set once, before the context opens)
  int front;               // how far the owner will get before a helper could finish a claim made now (it rises)
  int done;                // words finished by helpers (atomic)
  int ntrunc;              // rows cut short by the end of the stream (atomic), listed in the context's trunc array
  int err;                 // REST_CTX_* bits met by the gatherers (atomic)
  int pad[3];
};
static_assert(sizeof(ShareDesc) == 64, "one descriptor per 64 bytes");
constexpr int kShareMargin = 2;         // rounds (a word per warp) an owner gets through while a helper finishes one claim
constexpr int kShareRows = 512;         // candidate caps up to this never share (a block has a warp per word)
// Sharing costs every call a few microseconds (zeroing the counters, a grid of at least one block
// per SM, the look-outs), which the occasional long list must win back.  Measured on 100 M-token
// datastores: with a candidate cap of 20000 it pays from two contexts on (2: 38 -> 31 us,
// 16: 94 -> 50 us), with a cap of 5000 only from about 64 contexts on (2: 20 -> 26 us, 32: 31 ->
// 34 us, 64: equal, 128: 48 -> 43 us); a single context never shares.
constexpr int kShareMinContexts = 2;
constexpr int kShareMaxContexts = 1024;
constexpr int kShareLongCap = 8192;     // candidate caps from here on share whatever the batch
constexpr int kShareFromContexts = 48;  // shorter caps share from this many contexts on
static bool wants_share(int K, int B) {
  return K > kShareRows && B >= kShareMinContexts && B <= kShareMaxContexts &&
         (K >= kShareLongCap || B >= kShareFromContexts);
}  // calls with more contexts do not share (and take the batched path anyway)
constexpr int kShareHdr = 16;           // int32 counters ahead of the per-context arrays: [0] blocks started, [1] contexts past their gather
constexpr int kHelperPolls = 20000;     // idle polls (>= 200 ns each) after which a helper leaves
constexpr int kOwnerPolls = 1 << 20;    // polls after which an owner gives up on claimed chunks (REST_CTX_INTERNAL)

// Scratch of the shared gather for B contexts: counters, a state word and a descriptor per
// context (this part is zeroed before every launch), then the lists of short rows and the bitmaps.
struct ShareLayout {
  size_t ready, desc, zeroed_bytes, trunc, bm, bytes;     // byte offsets
};
static ShareLayout share_layout(int B, int m, int nwords) {
  ShareLayout l;
  const size_t bpad = ((size_t)B + 31) / 32 * 32;
  l.ready = kShareHdr * sizeof(int32_t);
  l.desc = l.ready + bpad * sizeof(int32_t);
  l.zeroed_bytes = l.desc + (size_t)B * sizeof(ShareDesc);
  l.trunc = l.zeroed_bytes;
  l.bm = l.trunc + (size_t)B * kMaxTrunc * sizeof(uint32_t);
  l.bytes = l.bm + (size_t)B * m * nwords * sizeof(uint32_t);
  return l;
}

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
// `run` (STRICT = false only): what the probes of the search tell about the END of the run of
// equal slots, for free: run[0] = the last probed slot that compared equal (-1: none), run[1] =
// the first probed slot that compared greater (in: the slot the search may assume greater,
// normally hi).  The first slot that compares greater lies in (run[0], run[1]].
//
// A = 32: every round all 32 lanes probe (fewest dependent rounds: the single-context path).
// A < 32: only the first WIDE rounds are 32 wide (a search over the whole array: their probe
// positions are the top of a fixed 33-ary tree, the same for every context, and stay in L2); the rounds
// below them, whose probes go to DRAM, use A lanes (A probes cut the interval into A + 1
// parts), which costs more dependent rounds but far fewer random DRAM reads per search.
template <typename SaT, bool STRICT, int A = 32, int WIDE = kWideRounds>
__device__ int64_t warp_first_true(const int32_t* __restrict__ T, const SaT* __restrict__ sa,
                                   int64_t n_tokens, int64_t lo, int64_t hi, const int (&q)[16],
                                   int n, int lane, bool& eq, bool& bad, int64_t* run = nullptr) {
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
    if (!STRICT && run) {
      // outcomes are monotone along the probes: smaller ... equal ... greater
      const unsigned eqb = __ballot_sync(kFull, c == 0 && lane <= last);
      const unsigned gtb = __ballot_sync(kFull, c > 0 && lane <= last);
      if (eqb) run[0] = max(run[0], __shfl_sync(kFull, pos, 31 - __clz(eqb)));
      if (gtb) run[1] = min(run[1], __shfl_sync(kFull, pos, __ffs(gtb) - 1));
    }
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
  if (!STRICT && run) {
    const unsigned eqb = __ballot_sync(kFull, (pos < hi) && c == 0);
    const unsigned gtb = __ballot_sync(kFull, (pos < hi) && c > 0);
    if (eqb) run[0] = max(run[0], lo + (int64_t)(31 - __clz(eqb)));
    if (gtb) run[1] = min(run[1], lo + (int64_t)(__ffs(gtb) - 1));
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

// Executed by a whole block of NT threads.  hist[0..nbins) holds counts; total >= need >= 1.
// Finds the largest bin b with sum(hist[k], k > b) < need; writes b and that sum (visible after
// the caller's next barrier).  scan: NT / 32 words of shared memory.
template <int NT>
__device__ __forceinline__ void block_threshold_desc(const uint32_t* hist, int nbins, uint32_t need, uint32_t* scan,
                                                     int* out_bin, uint32_t* out_above) {
  constexpr int NW = NT / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (nbins + NT - 1) / NT;        // bins per thread, from the top down
  const int top = nbins - 1 - tid * per;
  const int bot = max(0, top - per + 1);
  uint32_t sum = 0;
  for (int b = top; b >= bot; --b) sum += hist[b];
  uint32_t incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(kFull, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) scan[warp] = incl;
  __syncthreads();
  if (warp == 0) {                              // exclusive prefix over the warps' totals
    const uint32_t mine = lane < NW ? scan[lane] : 0u;
    uint32_t t = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(kFull, t, o);
      if (lane >= o) t += v;
    }
    if (lane < NW) scan[lane] = t - mine;
  }
  __syncthreads();
  const uint32_t excl = scan[warp] + incl - sum;
  if (excl < need && need <= excl + sum) {
    uint32_t acc = excl;
    for (int b = top; b >= bot; --b) {
      const uint32_t h = hist[b];
      if (acc + h >= need) { *out_bin = b; *out_above = acc; break; }
      acc += h;
    }
  }
}

struct Smem {
  int q[16];
  long long lb[17], ub[17];
  long long ub_from[17];       // >= 0: ub[n] is only known to lie in (ub_from[n] - 1, ub[n]]
  uint32_t small[5][kMaxM + 1];   // [c][d]: nodes of weight c = 1 ... 4 at depth d
  uint32_t big_total;          // nodes of weight >= 5
  int err;
  int bin_hi;
  uint32_t above_hi;
  int bin_lo;
  uint32_t above_lo;
  uint32_t nsel;
  uint32_t scan[32];           // warp totals of a block-wide prefix sum
  int ntrunc;
  int counted;                 // shared gathering: this context is counted as past its gather
  int help_b;                  // shared gathering: the context this block helps next
  int help_base, help_top;     // shared gathering: the words [base, top) of the block's current claim
  uint32_t trunc[kMaxTrunc];   // len << 16 | row: rows cut short by the end of the token stream
  uint32_t sel[kMaxN];         // depth << 16 | row
  uint32_t selcnt[kMaxN];
  uint32_t sorted[kMaxN];
  uint32_t sortedcnt[kMaxN];
  int par[kMaxN];
  uint32_t hist_hi[kHistHi];   // nodes of weight >= 5 by weight: exact below 1024, in steps of 32 above
  uint32_t hist_lo[kHistLo];   // inside the threshold bin: by depth (and the weight's low bits)
};

// Suffix-array range of the suffixes that start with the longest indexed prefix of q (n tokens):
// the bucket index is asked for q's first 2, 3, ... min(n, levels) tokens at once (four lanes
// per length read the four entries of that n-gram's group, one 128-byte line each) and the
// longest one stored wins.  Returns its length (0: none stored) and its range.
__device__ __forceinline__ int index_ngram_range(const rest::BucketIndex& idx, const int (&q)[16], int n,
                                                 int lane, int64_t n_slots, int64_t& lo, int64_t& hi) {
  const int level = 2 + (lane >> 2);
  const bool asks = lane < 4 * (rest::kIndexMaxLevel - 1) && level <= n && level <= idx.levels;
  unsigned long long key = (unsigned long long)(level - 1) << 62, k = rest::kIndexEmptyKey;
#pragma unroll
  for (int t = 0; t < rest::kIndexMaxLevel; ++t)
    if (t < level) key |= (unsigned long long)(uint32_t)q[t] << (t * idx.token_bits);
  long long l = -1, h = -1;
  if (asks) {
    const unsigned long long* e = idx.table + (size_t)rest::index_group_of(key, idx.group_mask) * 16 + (lane & 3) * 4;
    k = __ldg(e);
    l = (long long)__ldg(e + 1);
    h = (long long)__ldg(e + 2);
  }
  const unsigned hit = __ballot_sync(kFull, asks && k == key && l >= 0 && h > l && h <= n_slots);
  if (hit == 0) return 0;
  const int src = 31 - __clz(hit);           // the highest lane that hit asks for the longest n-gram
  lo = __shfl_sync(kFull, l, src);
  hi = __shfl_sync(kFull, h, src);
  return 2 + (src >> 2);
}

// Rows in bitmap word w whose continuation is shorter than d tokens (they end a run like any
// row that starts a node, but are no node at depth d themselves).  The list is almost always
// empty: only matches within m tokens of the end of the stream are cut short.
__device__ __forceinline__ uint32_t cut_short_mask(const Smem& s, int ntrunc, int d, int w) {
  uint32_t t = 0;
  for (int k = 0; k < ntrunc; ++k) {
    const uint32_t e = s.trunc[k];
    const int j = (int)(e & 0xFFFFu), len = (int)(e >> 16);
    if ((j >> 5) == w && len < d) t |= 1u << (j & 31);
  }
  return t;
}

// TP = false: the single-context path, tuned for the fewest dependent reads.  TP = true: the
// batched path, for calls with more contexts than the GPU holds at once; the same results by
// fewer random DRAM reads per context (see phase 1).
// PART: kWhole = search and build in one launch; kSearch = phase 1 only (writes match_n and
// match_range, the defaults of every output slot, and the context's index into one of two
// lists); kBuild = phases 2-4 for the contexts of one list; kRetrieve = phase 1 alone, nothing
// but match_n, match_range and status written (rest_retrieve); kFromRuns = phases 2-4 over rows
// that the caller hands in as sorted runs, merged first (rest_draft_from_runs); kWholeShare =
// kWhole with shared gathering (see ShareDesc; the grid may hold more blocks than contexts).
enum { kWhole = 0, kSearch = 1, kBuild = 2, kRetrieve = 3, kFromRuns = 4, kWholeShare = 5 };

// Three-way comparison of two candidate rows (tokens as unsigned integers; a row that is a
// proper prefix of the other sorts first).
__device__ __forceinline__ int compare_rows(const int32_t* __restrict__ y, int ylen, const int (&x)[kMaxM], int xlen) {
  const int lim = ylen < xlen ? ylen : xlen;
  for (int k = 0; k < lim; ++k) {
    const uint32_t a = (uint32_t)y[k], b = (uint32_t)x[k];
    if (a != b) return a < b ? -1 : 1;
  }
  return ylen == xlen ? 0 : (ylen < xlen ? -1 : 1);
}
// ---- gather rows, common-prefix lengths, node-start bitmap words -----------------------------
// Executed by one warp, for the context whose matched range is [lo, lo + cnt), of which Kp rows
// are taken, behind a match of n_win tokens.  Bitmap word w covers candidate rows 32 w ... 32 w + 31;
// the warp takes words first_word, first_word + stepw, ... below end_word (and below *limit,
// when given; see the shared gather).  The suffix-array entries of the warp's next word travel while the rows of the
// current one do.
// Slot 0 of the warp is the row before its first row, slot l + 1 the row of lane l.  A load
// instruction fetches two slots, 16 columns each (lane = 16 * slot parity + column): the
// lanes of a row read consecutive tokens, so an instruction touches two rows (a few cache
// lines) instead of 32.  A token is compared with the token above it (the same column of the
// slot before: the other half-warp of the same load, or of the load before) right where it
// sits; a ballot turns the "equal" and "smaller" outcomes of each load into bit strings, and
// lane l cuts the 16 bits of its row out of them: the number of leading equal columns is the
// common prefix.
// sb, sl: the warp's slot tables (34 entries each).  bm_out[d * a.nwords + w]: the words.  Rows
// cut short by the end of the stream are appended to trunc_out (counter ntrunc_out), problems
// OR-ed into err_out (all three in shared or global memory); pc[j], j < pc_rows, receives the
// suffix position of row j.
template <typename SaT, int PART>
__device__ __forceinline__ void gather_words(const DraftArgs& a, int b, const int32_t** sb, int* sl, int lane,
                                             int64_t lo, int64_t cnt, int Kp, int n_win, int first_word,
                                             int stepw, int end_word, uint32_t* bm_out, int* ntrunc_out,
                                             uint32_t* trunc_out, int* err_out, long long* pc, int pc_rows,
                                             const int* limit = nullptr, int limit_floor = 0,
                                             int* front_out = nullptr) {
  const int m = a.m, nwords = a.nwords;
  const int nw = end_word;
  const int64_t n_tokens = a.n_tokens;
  const SaT* __restrict__ sa = static_cast<const SaT*>(a.sa);
  // where the rows' tokens live: the token stream, or the caller's rows of this context
  const int32_t* __restrict__ Trow = PART == kFromRuns ? a.T + (int64_t)b * a.R * a.Kr * m : a.T;
  // where row j comes from: the suffix-array entry of its sampled slot lo + floor(j cnt / K), or
  // (rows handed in as runs) its place in the caller's row array, through the merged order.
  // floor(j cnt / K) = j floor(cnt / K) + floor(j (cnt mod K) / K), and j (cnt mod K) < 2^30: one
  // 64-bit division per context, a 32-bit one per row.
  const uint32_t* ord = PART == kFromRuns ? a.order + (int64_t)b * a.kcap : nullptr;
  const bool strided = PART != kFromRuns && cnt > (int64_t)a.K && a.sample_mode == REST_SAMPLE_STRIDED;
  const uint32_t uK = (uint32_t)a.K;
  const unsigned long long q1 = strided ? (unsigned long long)cnt / uK : 1ull;
  const uint32_t r1 = strided ? (uint32_t)((unsigned long long)cnt % uK) : 0u;
  auto entry_of = [&](int j) -> int64_t {
    if constexpr (PART == kFromRuns) return (int64_t)ord[j];
    else return (int64_t)__ldg(sa + lo + (int64_t)((unsigned long long)j * q1 + (unsigned long long)(((uint32_t)j * r1) / uK)));
  };
  // start of the row's tokens (relative to Trow) and its length; `bad` when the entry is out of range
  auto row_place = [&](int64_t& p, int64_t& base, int& len, bool& bad) {
    if constexpr (PART == kFromRuns) {
      if (p < 0 || p >= (int64_t)a.R * a.Kr) { bad = true; p = 0; }
      len = bad ? 0 : min(max(a.row_len[(int64_t)b * a.R * a.Kr + p], 0), m);
      p *= m;
      base = p;
    } else {
      if (p < 0 || p >= n_tokens) { bad = true; p = 0; }
      base = p + n_win;
      const int64_t rem_t = n_tokens - base;
      len = bad ? 0 : (int)(rem_t < 0 ? 0 : (rem_t > m ? m : rem_t));
    }
  };
  // the entries of word w: this lane's row, and (lane 0) the row before the word
  auto entries_of = [&](int w, int64_t& p, int64_t& pp) {
    p = 0; pp = 0;
    if (w >= nw) return;
    const int j = w * 32 + lane;
    if (j < Kp) p = entry_of(j);
    if (lane == 0 && w > 0) pp = entry_of(w * 32 - 1);
  };
  int w = first_word;
  int64_t p = 0, pp = 0;
  entries_of(w, p, pp);
  const int half = lane >> 4, col = lane & 15;
  if (lane == 0) { sl[33] = 0; sb[33] = Trow; }     // slot 33 does not exist
  // columns past a row's end read as a value no token has (tokens are below 2^31), different
  // for neighbouring slots: they never compare equal to anything above or below them
  const uint32_t pad = 0x80000000u | (uint32_t)half;
  // limit: words from max(*limit, limit_floor) on belong to somebody else (*limit only ever
  // falls); read one word ahead.  front_out: where this warp tells helpers how far it will be
  // by the time a claim made now could be finished (a hint: claims below it are not worth making)
  int stop = limit ? max(*reinterpret_cast<const volatile int*>(limit), limit_floor) : nw;
  while (w < nw && w < stop) {
    const int stop_next = limit ? max(*reinterpret_cast<const volatile int*>(limit), limit_floor) : nw;
    if (front_out && lane == 0) *reinterpret_cast<volatile int*>(front_out) = w + kShareMargin * stepw;
    const int jbase = w * 32;
    const int j = jbase + lane;
    const bool valid = j < Kp;
    bool bad = false;
    int len = 0;
    int64_t base = 0;
    if (valid) {
      row_place(p, base, len, bad);
      if (j < pc_rows) pc[j] = p;
    }
    int plen = __shfl_up_sync(kFull, len, 1);
    if (lane == 0) {
      plen = 0;
      int64_t pbase = 0;
      if (j > 0) row_place(pp, pbase, plen, bad);   // the row before belongs to another warp
      sb[0] = Trow + pbase; sl[0] = plen;
    }
    const int lim = min(len, plen);
    sb[lane + 1] = Trow + base; sl[lane + 1] = len;
    __syncwarp();
    uint32_t vals[kRowLoads];
#pragma unroll
    for (int i = 0; i < kRowLoads; ++i) {
      const int r = 2 * i + half;
      vals[i] = col < sl[r] ? (uint32_t)__ldg(sb[r] + col) : pad;
    }
    // the next word's suffix-array entries travel while this word's rows do
    const int wn = w + stepw;
    int64_t p_next, pp_next;
    entries_of(wn, p_next, pp_next);
    uint32_t my_eq = 0, my_lt = 0, other_prev = 0;     // lane i keeps the bit strings of load i
#pragma unroll
    for (int i = 0; i < kRowLoads; ++i) {
      const uint32_t other = __shfl_xor_sync(kFull, vals[i], 16);   // same column, other slot of this load
      const uint32_t above = half ? other : other_prev;             // the slot before this one
      const uint32_t eq = __ballot_sync(kFull, vals[i] == above);
      const uint32_t lt = __ballot_sync(kFull, above < vals[i]);
      if (lane == i) { my_eq = eq; my_lt = lt; }
      other_prev = other;
    }
    // this lane's row is slot lane + 1: load (lane + 1) / 2, upper half of the word when odd
    const int slot = lane + 1, sh = (slot & 1) << 4;
    const uint32_t eqf = (__shfl_sync(kFull, my_eq, slot >> 1) >> sh) & 0xFFFFu;
    const uint32_t ltf = (__shfl_sync(kFull, my_lt, slot >> 1) >> sh) & 0xFFFFu;
    int lcp = __ffs((int)(~eqf | 0x10000u)) - 1;       // leading equal columns (padding never matches: at most lim)
    if (!valid || j == 0) lcp = 0;
    if (valid && j > 0) {
      // the first differing column decides the order; when one row is a prefix of the
      // other the shorter one must come first
      const bool ordered = lcp < lim ? ((ltf >> lcp) & 1u) != 0u : plen <= len;
      if (!ordered) bad = true;
    }
    if (valid && len < m) {        // cut short by the end of the stream: at most m such rows exist
      const int at = atomicAdd(ntrunc_out, 1);
      if (at < kMaxTrunc) trunc_out[at] = ((uint32_t)len << 16) | (uint32_t)j;
      else atomicOr(err_out, REST_CTX_INTERNAL);
    }
    uint32_t myword = 0;
#pragma unroll
    for (int d = 1; d <= kMaxM; ++d) {
      const uint32_t wd = __ballot_sync(kFull, !valid || lcp < d);
      if (lane == d - 1) myword = wd;
    }
    if (lane < m) bm_out[lane * nwords + w] = myword;
    if (__any_sync(kFull, bad) && lane == 0) atomicOr(err_out, REST_CTX_BAD_DATASTORE);
    __syncwarp();                  // the slot tables are rewritten by the next word
    w = wn; p = p_next; pp = pp_next;
    stop = stop_next;
  }
}

// Executed by a whole block: works on the words that other contexts offer until none is left to
// claim (no waiting).  `start`: where the block begins its look-out.  only_if_all_started: do
// nothing while contexts of the launch still wait for an SM (this block had better finish and
// make room).  Warp 0 looks out and claims (a context whose words are all claimed costs it one
// read, no barrier); the block meets only over a claim that succeeded.
template <typename SaT, int NT>
__device__ __forceinline__ void share_help_pass(const DraftArgs& a, Smem& s, const int32_t** sb, int* sl, int start,
                                                bool only_if_all_started) {
  constexpr int NW = NT / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int B = a.B, bpad = (B + 31) & ~31;
  int cur = -1;                        // the context the block worked on last (its fields are still at hand)
  int64_t lo = 0, cnt = 0;
  int Kp = 0, n_win = 0, nw = 0;
  int finished = 0;                    // words of the round before, not yet counted
  bool allowed = !only_if_all_started;
  for (;;) {
    if (warp == 0) {
      if (finished && lane == 0) atomicAdd(&a.sh_desc[cur].done, finished);
      int found = -1, base = 0, top = 0;
      if (!allowed) allowed = *reinterpret_cast<volatile int32_t*>(a.sh_hdr) >= B;
      int prefer = cur;
      for (int tries = 0; allowed && tries <= B && found < 0; ++tries) {
        int cand = prefer;
        prefer = -1;
        if (cand < 0) {
          for (int k = 0; k < bpad && cand < 0; k += 32) {
            int bb = (start & ~31) + k + lane;
            if (bb >= bpad) bb -= bpad;
            const int st = bb < B ? *reinterpret_cast<volatile int32_t*>(a.sh_ready + bb) : 0;
            const unsigned open = __ballot_sync(kFull, st == 1);
            if (open) cand = __shfl_sync(kFull, bb, __ffs(open) - 1);
          }
          if (cand < 0) break;
        }
        ShareDesc* dsc = a.sh_desc + cand;
        // take the NW words below `back` (fewer when that reaches under the floor, the words
        // that must be the owner's own)
        // ... and none at all when the owner will be there before this block could finish them: it
        // would only have to wait for them
        const int floor = *reinterpret_cast<volatile int*>(&dsc->floor);
        const int front = *reinterpret_cast<volatile int*>(&dsc->front);
        int hi = *reinterpret_cast<volatile int*>(&dsc->back);
        if (hi > floor && hi - NW >= front) {
          if (lane == 0) hi = atomicSub(&dsc->back, NW);
          hi = __shfl_sync(kFull, hi, 0);
        } else {
          hi = 0;
        }
        if (hi > floor) { found = cand; base = max(floor, hi - NW); top = hi; }
        else if (lane == 0) *reinterpret_cast<volatile int32_t*>(a.sh_ready + cand) = 2;     // every word is taken
      }
      __threadfence();
      if (lane == 0) { s.help_b = found; s.help_base = base; s.help_top = top; }
    }
    __syncthreads();
    const int found = s.help_b, base = s.help_base, end = s.help_top;
    __syncthreads();
    finished = 0;
    if (found < 0) break;
    if (found != cur) {
      const ShareDesc* dsc = a.sh_desc + found;
      lo = __ldcg(&dsc->lo); cnt = __ldcg(&dsc->cnt);
      Kp = __ldcg(&dsc->Kp); n_win = __ldcg(&dsc->n_win); nw = __ldcg(&dsc->nw);
      cur = found;
    }
    // a descriptor that makes no sense is left to its owner (the words claimed from it stay
    // uncounted: its owner reports the context as failed)
    const bool sane = Kp > 0 && Kp <= a.kcap && cnt >= (int64_t)Kp && lo >= 0 && lo + cnt <= a.n_sa &&
                      n_win >= 1 && nw == ((Kp + 31) >> 5) && base >= 0 && base < end && end <= nw;
    if (!sane) {
      if (tid == 0) *reinterpret_cast<volatile int32_t*>(a.sh_ready + found) = 2;
      cur = -1;
      continue;
    }
    ShareDesc* dsc = a.sh_desc + found;
    gather_words<SaT, kWholeShare>(a, found, sb, sl, lane, lo, cnt, Kp, n_win, base + warp, NW, end,
                                   a.sh_bm + (int64_t)found * a.m * a.nwords, &dsc->ntrunc,
                                   a.sh_trunc + (int64_t)found * kMaxTrunc, &dsc->err, nullptr, 0);
    __threadfence();                   // the words before the count
    __syncthreads();
    finished = end - base;
  }
}

// The work of one block on its context (blockIdx.x, or the blockIdx.x-th of a list).
template <typename SaT, bool TP, int NT, int PART>
__device__ __forceinline__ void draft_block(const DraftArgs& a, unsigned char* smem_raw) {
  constexpr int NW = NT / 32;
  static_assert(NT % 32 == 0 && NT >= 128, "whole warps; enough threads for the set-up loops");
  Smem& s = *reinterpret_cast<Smem*>(smem_raw);
  // per warp: token address and length of its 33 slots (the row before the
  // warp's first one, then its 32 rows); the suffix positions of the first rows (phase 4 reads
  // the kept nodes' tokens through them); then the block's bitmaps
  long long* slot_base = reinterpret_cast<long long*>(smem_raw + sizeof(Smem));            // [NW][34]
  long long* pcache = slot_base + NW * 34;                                                  // [pcache_rows]
  int* slot_len = reinterpret_cast<int*>(pcache + a.pcache_rows);                           // [NW][34]
  uint32_t* bm = reinterpret_cast<uint32_t*>(slot_len + NW * 34);                           // [m][nwords]
  // nodes of weight >= 5 met by the first pass over the bitmaps: (depth << 16 | row) and weight
  // (the 32-bit arrays first, then the 16-bit ones: every array is aligned to its element size)
  uint32_t* big_dj = bm + a.m * a.nwords;                                                   // [bigcap]
  uint16_t* jump = reinterpret_cast<uint16_t*>(big_dj + a.bigcap);                          // [m][nwords]
  uint16_t* tiecnt = jump + a.m * a.nwords;                                                 // [nwords]
  uint16_t* big_c = tiecnt + a.nwords;                                                      // [bigcap]

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
  const int64_t n_sa = a.n_sa;          // slots of the suffix array (searches), n_tokens bounds positions
  const int clen = a.ctx_len[b];
  const int32_t* ctx = PART == kFromRuns ? nullptr : a.ctx + (int64_t)b * a.ctx_stride;
  // read early, beside the context: whether the bucket index may be used (not when its build
  // met a suffix-array entry or a token out of range)
  const uint32_t index_unusable =
      (PART != kBuild && PART != kFromRuns && a.idx.first != nullptr) ? __ldg(a.idx.unusable) : 1u;

  // Unused-slot defaults; thread i owns slots i, i + NT, ... for the whole kernel (a build
  // launch finds them written by the search launch).
  auto write_defaults = [&]() {
    for (int i = tid; i < N; i += NT) {
      int64_t o = (int64_t)b * N + i;
      a.tokens[o] = -1; a.parents[o] = -1; a.depth[o] = 0; a.pos_ids[o] = clen;
      for (int w = 0; w < Wm; ++w) a.mask[o * Wm + w] = (w == (i >> 5)) ? (1u << (i & 31)) : 0u;
      if (a.node_count) a.node_count[o] = 0;
    }
  };
  auto report_empty = [&]() {                      // by thread 0, after a barrier
    a.status[b] = s.err;
    if (a.n_nodes) a.n_nodes[b] = 0;
    if (a.match_n) a.match_n[b] = 0;
    if (a.match_range) { a.match_range[2 * b] = 0; a.match_range[2 * b + 1] = 0; }
  };
  if constexpr (PART == kWhole || PART == kWholeShare || PART == kSearch || PART == kFromRuns) write_defaults();
  const int nq = min(a.n_max, max(clen, 0));   // context tokens that can take part
  if (tid == 0) { s.err = 0; s.big_total = 0; s.nsel = 0; s.ntrunc = 0; s.counted = 0; }
  if (tid < 17) { s.lb[tid] = 0; s.ub[tid] = 0; s.ub_from[tid] = -1; }
  if (tid < 5 * (kMaxM + 1)) (&s.small[0][0])[tid] = 0;
  if constexpr (PART != kSearch && PART != kRetrieve) {
    for (int i = tid; i < kHistHi; i += NT) s.hist_hi[i] = 0;
    for (int i = tid; i < kHistLo; i += NT) s.hist_lo[i] = 0;
  }
  __syncthreads();
  int n_win = 0;
  if constexpr (PART == kBuild) {
    n_win = a.match_n[b];
    if (tid == 0) { s.lb[n_win] = a.match_range[2 * b]; s.ub[n_win] = a.match_range[2 * b + 1]; }
    __syncthreads();
  } else if constexpr (PART == kFromRuns) {
    // The rows arrive as R runs, each in lexicographic order (the rows of one suffix-array
    // range are).  Position of row i of run r in the merged order: i, plus for every other run
    // the number of its rows that sort before this one (equal rows: the lower run first), found
    // by bisection.  Runs that are not in order leave slots of the order unwritten, which the
    // gather below reports as a bad datastore.
    const int R = a.R, Kr = a.Kr;
    const int32_t* nrun = a.run_rows + (int64_t)b * R;
    const int32_t* rows = T + (int64_t)b * R * Kr * m;
    const int32_t* lens = a.row_len + (int64_t)b * R * Kr;
    uint32_t* ord = a.order + (int64_t)b * a.kcap;
    int total = 0;
    for (int r = 0; r < R; ++r) total += min(max(nrun[r], 0), Kr);
    for (int x = tid; x < a.kcap; x += NT) ord[x] = 0xFFFFFFFFu;
    __syncthreads();
    for (int flat = tid; flat < R * Kr; flat += NT) {
      const int r = flat / Kr, i = flat - r * Kr;
      if (i >= min(max(nrun[r], 0), Kr)) continue;
      int mine[kMaxM];
      const int mylen = min(max(lens[flat], 0), m);
#pragma unroll
      for (int k = 0; k < kMaxM; ++k) mine[k] = k < mylen ? rows[(int64_t)flat * m + k] : 0;
      int rank = i;
      for (int r2 = 0; r2 < R; ++r2) {
        if (r2 == r) continue;
        int lo2 = 0, hi2 = min(max(nrun[r2], 0), Kr);
        while (lo2 < hi2) {
          const int mid = (lo2 + hi2) >> 1, f2 = r2 * Kr + mid;
          const int c = compare_rows(rows + (int64_t)f2 * m, min(max(lens[f2], 0), m), mine, mylen);
          if (c < 0 || (c == 0 && r2 < r)) lo2 = mid + 1; else hi2 = mid;
        }
        rank += lo2;
      }
      if (rank < a.kcap) ord[rank] = (uint32_t)flat;
    }
    if (tid == 0) { s.lb[0] = 0; s.ub[0] = total < a.kcap ? total : a.kcap; }
    __syncthreads();
    if (total == 0) {
      if (tid == 0) report_empty();
      return;
    }
  } else {
  if (tid < nq) {
    int t = ctx[clen - nq + tid];
    s.q[tid] = t;
    if (t < 0 || (uint32_t)t >= a.vocab) atomicOr(&s.err, REST_CTX_BAD_TOKEN);
  }
  __syncthreads();
  if (s.err != 0 || nq < a.n_min) {
    if (tid == 0) report_empty();
    return;
  }

  // ---- phase 1: search --------------------------------------------------------------
  // the range of every suffix length, one warp each (lb = ub: no match)
  constexpr int kArity = TP ? kTpArity : 32;
  const bool have_index = index_unusable == 0u;
  auto lower_bound_of = [&](int n) {     // executed by one whole warp
    int q[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) q[k] = (k < n) ? s.q[nq - n + k] : 0;
    bool bad = false, eq = false;
    int64_t lb;
    // the end of the run of matches: first slot after lb that compares greater.  The probes of
    // the lower bound bracket it for free (last probed slot seen equal, first seen greater).
    // Only the longest matching length needs its end, so a bracket that is not settled yet is
    // left as it is: the search inside it runs after the barrier, for the winner alone.
    auto finish = [&](int64_t lb_, int64_t end, int64_t (&run)[2]) {
      if (lane != 0) return;
      s.lb[n] = lb_;
      s.ub[n] = lb_;                       // no match: empty range
      if (eq && lb_ < end) {
        const int64_t from = (run[0] > lb_ ? run[0] : lb_) + 1;
        s.ub[n] = run[1];                  // > lb_: a match
        if (from < run[1]) s.ub_from[n] = from;
      }
    };
    if (have_index) {
      // every suffix that starts with the query's first token lies in [f0, f1); when the index
      // also stores the query's first two, three or four tokens, every suffix that starts with
      // those lies in [lo0, hi0).  Slot hi0 (or the end of the array) compares greater than the query.
      int64_t lo0 = __ldg(a.idx.first + q[0]), hi0 = __ldg(a.idx.first + q[0] + 1);
      lo0 = lo0 < 0 ? 0 : (lo0 > n_sa ? n_sa : lo0);
      hi0 = hi0 < lo0 ? lo0 : (hi0 > n_sa ? n_sa : hi0);
      if (n == 1) {                       // the first-token range is the answer
        if (lane == 0) { s.lb[1] = lo0; s.ub[1] = hi0; }
        return;
      }
      int64_t plo = 0, phi = 0;
      const int found = index_ngram_range(a.idx, q, n, lane, n_sa, plo, phi);
      if (found > 0 && plo >= lo0 && phi <= hi0) {
        if (found == n) {                 // the n-gram's own range is the answer
          if (lane == 0) { s.lb[n] = plo; s.ub[n] = phi; }
          return;
        }
        lo0 = plo; hi0 = phi;
      }
      int64_t run[2] = {-1, hi0};
      lb = warp_first_true<SaT, false, kArity, 0>(T, sa, n_tokens, lo0, hi0, q, n, lane, eq, bad, run);
      finish(lb, hi0, run);
    } else {
      int64_t run[2] = {-1, n_sa};
      lb = warp_first_true<SaT, false, kArity>(T, sa, n_tokens, 0, n_sa, q, n, lane, eq, bad, run);
      finish(lb, n_sa, run);
    }
    if (__any_sync(kFull, bad) && lane == 0) atomicOr(&s.err, REST_CTX_BAD_DATASTORE);
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
  if (n_win != 0 && s.ub_from[n_win] >= 0) {     // the same for the whole block
    // the end of the winner's run: first slot in [ub_from, ub) that compares greater, else ub
    // (the new ub is above lb like the old one, so warps still picking n_win read the same answer)
    if (warp == 0) {
      int q[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) q[k] = (k < n_win) ? s.q[nq - n_win + k] : 0;
      bool bad = false, eq = false;
      const int64_t ub = warp_first_true<SaT, true, kArity, 0>(T, sa, n_tokens, s.ub_from[n_win], s.ub[n_win],
                                                                q, n_win, lane, eq, bad);
      if (__any_sync(kFull, bad) && lane == 0) atomicOr(&s.err, REST_CTX_BAD_DATASTORE);
      __syncwarp();
      if (lane == 0) s.ub[n_win] = ub;
    }
    __syncthreads();
  }
  if (s.err != 0 || n_win == 0) {
    if (tid == 0) report_empty();
    return;
  }
  }  // PART != kBuild
  const int64_t lo = s.lb[n_win], hi = s.ub[n_win];
  const int64_t cnt = hi - lo;
  if constexpr (PART == kRetrieve) {
    if (tid == 0) {
      a.status[b] = 0; a.match_n[b] = n_win;
      a.match_range[2 * b] = lo; a.match_range[2 * b + 1] = hi;
    }
    return;
  }
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
  // where the rows' tokens live: the token stream, or the caller's rows of this context
  const int32_t* __restrict__ Trow = PART == kFromRuns ? T + (int64_t)b * a.R * a.Kr * m : T;
  const int nwords = a.nwords;
  const int nw = (Kp + 31) >> 5;            // bitmap words that hold rows

  // ---- phase 2: gather rows, common-prefix lengths, node-start bitmaps --------------------
  const int32_t** my_sb = reinterpret_cast<const int32_t**>(slot_base + warp * 34);
  int* my_sl = slot_len + warp * 34;
  bool shared_gather = false;
  int own_words = nw;                  // bitmap words whose rows this block read itself
  // worth it with more words than warps, and with words beyond the rows whose positions stay here
  if constexpr (PART == kWholeShare) shared_gather = Kp > max(a.share_rows, NT) && nw > ((a.pcache_rows + 31) >> 5);
  if (!shared_gather) {
    // warp w takes words w, w + NW, ...
    gather_words<SaT, PART>(a, b, my_sb, my_sl, lane, lo, cnt, Kp, n_win, warp, NW, nw, bm, &s.ntrunc,
                            s.trunc, &s.err, pcache, a.pcache_rows);
    if constexpr (PART == kWholeShare) {
      if (tid == 0) { atomicAdd(a.sh_hdr + 1, 1); s.counted = 1; }     // this context offers nothing
      // its own rows read, the block works on the rows that other contexts offer right now (the
      // contexts that hold the call up) before it goes on with its own, smaller tree
      share_help_pass<SaT, NT>(a, s, my_sb, my_sl, b, true);
    }
  } else {
    // offer the end of the list to every idle block of the launch and work up from its start
    ShareDesc* dsc = a.sh_desc + b;
    const int floor = (a.pcache_rows + 31) >> 5;     // the rows whose positions phase 4 wants cached stay here
    if (tid == 0) {
      dsc->lo = lo; dsc->cnt = cnt; dsc->Kp = Kp; dsc->n_win = n_win; dsc->nw = nw;
      dsc->floor = floor; dsc->back = nw;
      __threadfence();
      *reinterpret_cast<volatile int32_t*>(a.sh_ready + b) = 1;
    }
    __syncthreads();                                 // `back` is set before any warp looks at it
    gather_words<SaT, PART>(a, b, my_sb, my_sl, lane, lo, cnt, Kp, n_win, warp, NW, nw, bm, &s.ntrunc,
                            s.trunc, &s.err, pcache, a.pcache_rows, &dsc->back, floor, warp == 0 ? &dsc->front : nullptr);
    __syncthreads();
    if (tid == 0) {
      // close: what the helpers hold now is all they will ever hold
      int from = atomicExch(&dsc->back, 0);
      from = max(floor, min(from, nw));
      *reinterpret_cast<volatile int32_t*>(a.sh_ready + b) = 2;
      atomicAdd(a.sh_hdr + 1, 1); s.counted = 1;
      int polls = 0;
      while (*reinterpret_cast<volatile int*>(&dsc->done) < nw - from && polls < kOwnerPolls) { __nanosleep(100); ++polls; }
      __threadfence();
      int e = *reinterpret_cast<volatile int*>(&dsc->err);
      if (*reinterpret_cast<volatile int*>(&dsc->done) < nw - from) e |= REST_CTX_INTERNAL;
      if (e) atomicOr(&s.err, e);
      s.help_base = from;
      s.help_top = min(max(*reinterpret_cast<volatile int*>(&dsc->ntrunc), 0), kMaxTrunc);
    }
    __syncthreads();
    own_words = s.help_base;
    if (s.err == 0) {
      // the helpers' part of the bitmaps, and the short rows they met
      const int from = own_words, nhelped = nw - from, ntr = s.help_top;
      const uint32_t* gbm = a.sh_bm + (int64_t)b * m * nwords;
#pragma unroll 4
      for (int i = tid; i < m * nhelped; i += NT) {
        const int d = i / nhelped, w = from + i - d * nhelped;
        bm[d * nwords + w] = __ldcg(gbm + d * nwords + w);
      }
      if (tid < ntr) {
        const int at = atomicAdd(&s.ntrunc, 1);
        if (at < kMaxTrunc) s.trunc[at] = __ldcg(a.sh_trunc + (int64_t)b * kMaxTrunc + tid);
        else atomicOr(&s.err, REST_CTX_INTERNAL);
      }
    }
  }
  // rows whose position phase 4 finds in shared memory (only rows this block read itself)
  const int pcache_rows = min(a.pcache_rows, own_words * 32);
  if (tid < m) bm[tid * nwords + ((Kp + 31) >> 5)] = kFull;   // sentinel past the last row
  __syncthreads();
  if (s.err != 0) {
    if (tid == 0) report_empty();
    return;
  }
  const int ntrunc = min(s.ntrunc, kMaxTrunc);

  // jump table: jump[w] = position of the first set bit in any word after w (0xFFFF: none).  A
  // warp takes a chunk of 32 words of a depth: a ballot of the non-empty words tells every lane
  // which lane behind it holds the next set bit.  With several chunks per depth, the first set
  // bit of every chunk is found first and, per depth, what the chunks behind a chunk hold.
  {
    const int last = (Kp + 31) >> 5;              // the sentinel word
    const int nchunk = (last >> 5) + 1;
    uint16_t* cmin = tiecnt;                      // [m][nchunk], free until phase 3c (16 nchunk <= nwords when nchunk > 1)
    const int step_d = NW / nchunk, step_c = NW - step_d * nchunk;     // a warp's next pair: NW further
    if (nchunk > 1) {                             // block-uniform
      int dd = warp / nchunk, c = warp - dd * nchunk;
#pragma unroll 2
      for (int pair = warp; pair < m * nchunk; pair += NW) {
        const int wi = c * 32 + lane;
        const uint32_t bits = wi <= last ? bm[dd * nwords + wi] : 0u;
        const unsigned nz = __ballot_sync(kFull, bits != 0u);
        const int v = (wi << 5) + __ffs(bits) - 1;
        const int first = __shfl_sync(kFull, v, nz ? __ffs(nz) - 1 : 0);
        if (lane == 0) cmin[pair] = (uint16_t)(nz ? first : 0xFFFF);
        dd += step_d; c += step_c;
        if (c >= nchunk) { c -= nchunk; ++dd; }
      }
      __syncthreads();
      // per depth: exclusive suffix minimum over the (at most 33) chunks
      for (int dd = warp; dd < m; dd += NW) {
        uint16_t* cm = cmin + dd * nchunk;
        int carry = 0xFFFF;
        for (int g0 = ((nchunk - 1) >> 5) << 5; g0 >= 0; g0 -= 32) {
          const int c = g0 + lane;
          int v = c < nchunk ? (int)cm[c] : 0xFFFF;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_down_sync(kFull, v, o);
            if (lane + o < 32) v = min(v, u);
          }
          v = min(v, carry);
          const int after = __shfl_down_sync(kFull, v, 1);
          if (c < nchunk) cm[c] = (uint16_t)(lane < 31 ? after : carry);
          carry = __shfl_sync(kFull, v, 0);
        }
      }
      __syncthreads();
    }
    int dd = warp / nchunk, c = warp - dd * nchunk;
#pragma unroll 2
    for (int pair = warp; pair < m * nchunk; pair += NW, dd += step_d, c += step_c) {
      if (c >= nchunk) { c -= nchunk; ++dd; }
      const int wi = c * 32 + lane;
      const uint32_t bits = wi <= last ? bm[dd * nwords + wi] : 0u;
      const unsigned nz = __ballot_sync(kFull, bits != 0u);
      const int v = (wi << 5) + __ffs(bits) - 1;
      const unsigned higher = nz & ~((2u << lane) - 1u);          // non-empty words behind this one in the chunk
      const int nextv = __shfl_sync(kFull, v, higher ? __ffs(higher) - 1 : lane);
      const int behind = nchunk > 1 ? (int)cmin[pair] : 0xFFFF;
      if (wi <= last) jump[dd * nwords + wi] = (uint16_t)(higher ? nextv : behind);
    }
  }
  __syncthreads();

  // The passes of phase 3 run over the pairs (depth d, bitmap word w).  In word w of depth d a
  // set bit marks a row that starts a node (unless the row is shorter than d) and the node's
  // weight is the distance to the next set bit.  Weights 1 to 4 are read off the bit pattern
  // (set bit, then 0 to 3 clear bits, then a set bit) for the whole word at once and counted
  // with one popcount each; only nodes of weight >= 5 are visited one by one.
  struct WordNodes { uint32_t c[5]; uint32_t big; };     // c[1..4]: node starts of that weight
  const int items = m * nw;
  auto word_nodes = [&](int d, int w) -> WordNodes {
    const uint32_t* row = bm + (d - 1) * nwords;
    const uint32_t S = row[w], nx = row[w + 1];
    uint32_t nodes = S;
    if (w == nw - 1 && (Kp & 31)) nodes &= (1u << (Kp & 31)) - 1u;     // bits past the last row
    if (ntrunc) nodes &= ~cut_short_mask(s, ntrunc, d, w);
    const unsigned long long W = (unsigned long long)S | ((unsigned long long)nx << 32);
    const uint32_t a1 = (uint32_t)(W >> 1), a2 = (uint32_t)(W >> 2), a3 = (uint32_t)(W >> 3), a4 = (uint32_t)(W >> 4);
    WordNodes r;
    r.c[0] = 0;
    r.c[1] = nodes & a1;
    uint32_t rest_ = nodes & ~a1;
    r.c[2] = rest_ & a2; rest_ &= ~a2;
    r.c[3] = rest_ & a3; rest_ &= ~a3;
    r.c[4] = rest_ & a4;
    r.big = rest_ & ~a4;
    return r;
  };
  // key of a node = weight << 5 | (16 - depth): larger key = better node.  First-level bin of a
  // node of weight >= 5: the weight itself below 1024, 1024 + weight / 32 above.
  auto key_of = [](int c, int d) -> uint32_t { return ((uint32_t)c << 5) | (uint32_t)(16 - d); };
  auto bin_of = [](int c) -> int { return c < 1024 ? c : 1024 + (c >> 5); };
  auto sub_of = [](int c, int d) -> int { return c < 1024 ? 16 - d : ((c & 31) << 5) | (16 - d); };

  // ---- phase 3a: counts of the light nodes, histogram of the others ------------------------
  // First the words: light nodes are counted, heavy nodes only listed (depth, row).  Then the
  // list, a thread per heavy node: its weight (distance to the next set bit) and its bin.  Short
  // dependent chains in both passes; a thread that walked its words' heavy nodes one by one,
  // weights included, held its warp up for a thousand cycles per word.
  {
    int d = tid / nw + 1, w = tid - (d - 1) * nw;
    const int step_d = NT / nw, step_w = NT - step_d * nw;          // a thread's next item: NT further
#pragma unroll 2
    for (int item = tid; item < items; item += NT) {
      const WordNodes wn = word_nodes(d, w);
#pragma unroll
      for (int c = 1; c <= 4; ++c)
        if (wn.c[c]) atomicAdd(&s.small[c][d], (uint32_t)__popc(wn.c[c]));
      uint32_t big = wn.big;
      if (big) {
        uint32_t at = atomicAdd(&s.big_total, (uint32_t)__popc(big));
        while (big) {
          if (at < (uint32_t)a.bigcap) big_dj[at] = ((uint32_t)d << 16) | (uint32_t)((w << 5) + __ffs(big) - 1);
          big &= big - 1;
          ++at;
        }
      }
      d += step_d; w += step_w;
      if (w >= nw) { w -= nw; ++d; }
    }
  }
  __syncthreads();
  const uint32_t big_total = s.big_total;
  const bool listed = big_total <= (uint32_t)a.bigcap;     // the list holds every heavy node
  if (listed) {
    for (uint32_t e = tid; e < big_total; e += NT) {
      const int d = (int)(big_dj[e] >> 16), j = (int)(big_dj[e] & 0xFFFFu);
      const int c = next_set(bm + (d - 1) * nwords, jump + (d - 1) * nwords, j) - j;
      big_c[e] = (uint16_t)c;
      atomicAdd(&s.hist_hi[bin_of(c)], 1u);
    }
  } else {
    // more heavy nodes than the list holds: this pass and the later ones walk the words again
    for (int item = tid; item < items; item += NT) {
      const int d = item / nw + 1, w = item - (d - 1) * nw;
      uint32_t big = word_nodes(d, w).big;
      const uint32_t* row = bm + (d - 1) * nwords;
      const uint16_t* jrow = jump + (d - 1) * nwords;
      while (big) {
        const int j = (w << 5) + __ffs(big) - 1;
        big &= big - 1;
        atomicAdd(&s.hist_hi[bin_of(next_set(row, jrow, j) - j)], 1u);
      }
    }
  }
  __syncthreads();

  // ---- phase 3b: threshold key t*, number of ties wanted ------------------------------------
  uint32_t tstar = 0;  // nodes with key > tstar are kept
  uint32_t r_tie = 0;  // plus the first r_tie nodes (by row) with key == tstar
  int c_tie = 0, d_tie = 0;
  if (big_total >= (uint32_t)N) {
    block_threshold_desc<NT>(s.hist_hi, kHistHi, (uint32_t)N, s.scan, &s.bin_hi, &s.above_hi);
    __syncthreads();
    const int bin_hi = s.bin_hi;
    if (listed) {
      for (uint32_t e = tid; e < big_total; e += NT) {
        const int c = (int)big_c[e];
        if (bin_of(c) == bin_hi) atomicAdd(&s.hist_lo[sub_of(c, (int)(big_dj[e] >> 16))], 1u);
      }
    } else
    for (int item = tid; item < items; item += NT) {
      const int d = item / nw + 1, w = item - (d - 1) * nw;
      uint32_t big = word_nodes(d, w).big;
      const uint32_t* row = bm + (d - 1) * nwords;
      const uint16_t* jrow = jump + (d - 1) * nwords;
      while (big) {
        const int j = (w << 5) + __ffs(big) - 1;
        big &= big - 1;
        const int c = next_set(row, jrow, j) - j;
        if (bin_of(c) == bin_hi) atomicAdd(&s.hist_lo[sub_of(c, d)], 1u);
      }
    }
    __syncthreads();
    block_threshold_desc<NT>(s.hist_lo, kHistLo, (uint32_t)N - s.above_hi, s.scan, &s.bin_lo, &s.above_lo);
    __syncthreads();
    const int sub = s.bin_lo;
    d_tie = 16 - (sub & 31);
    c_tie = bin_hi < 1024 ? bin_hi : (((bin_hi - 1024) << 5) | (sub >> 5));
    tstar = key_of(c_tie, d_tie);
    r_tie = (uint32_t)N - s.above_hi - s.above_lo;
  } else {
    // every node of weight >= 5 is kept; the lighter ones fill up by weight, then depth, then
    // row.  Every warp scans the 4 x 16 counts in that order for itself: lane l takes the
    // classes 2 l and 2 l + 1 (class k = weight 4 - k / 16 at depth k % 16 + 1).
    const uint32_t need = (uint32_t)N - big_total;
    const int k0 = 2 * lane, k1 = 2 * lane + 1;
    const int c0 = 4 - (k0 >> 4), d0 = (k0 & 15) + 1, c1 = 4 - (k1 >> 4), d1 = (k1 & 15) + 1;
    const uint32_t e0 = d0 <= m ? s.small[c0][d0] : 0u, e1 = d1 <= m ? s.small[c1][d1] : 0u;
    uint32_t incl = e0 + e1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t u = __shfl_up_sync(kFull, incl, o);
      if (lane >= o) incl += u;
    }
    const uint32_t before = incl - e0 - e1;
    const unsigned hit = __ballot_sync(kFull, incl >= need);      // need >= 1
    if (hit) {
      const int src = __ffs(hit) - 1;
      const uint32_t bsrc = __shfl_sync(kFull, before, src), e0s = __shfl_sync(kFull, e0, src);
      const bool first = bsrc + e0s >= need;
      const int k = 2 * src + (first ? 0 : 1);
      c_tie = 4 - (k >> 4); d_tie = (k & 15) + 1;
      tstar = key_of(c_tie, d_tie);
      r_tie = need - bsrc - (first ? 0u : e0s);
    }
  }

  // ---- phase 3c: collect the kept nodes -----------------------------------------------------
  // everything above the threshold now; the ties (same weight, same depth) by row order after a
  // prefix sum over the words of their depth
  auto keep = [&](int d, int j, int c) {
    const uint32_t slot = atomicAdd(&s.nsel, 1u);
    if (slot < (uint32_t)N) { s.sel[slot] = ((uint32_t)d << 16) | (uint32_t)j; s.selcnt[slot] = (uint32_t)c; }
  };
  // the first `take` nodes marked in `bits` (rows 32 w + bit) of depth d, weight c: one claim of slots
  auto keep_bits = [&](int d, int w, int c, uint32_t bits, uint32_t take) {
    uint32_t slot = atomicAdd(&s.nsel, take);
    for (; take > 0; --take, ++slot) {
      if (slot < (uint32_t)N) { s.sel[slot] = ((uint32_t)d << 16) | (uint32_t)((w << 5) + __ffs(bits) - 1); s.selcnt[slot] = (uint32_t)c; }
      bits &= bits - 1;
    }
  };
  auto tie_bits = [&](int w) -> uint32_t {         // tie candidates in word w of the tie depth
    const WordNodes wn = word_nodes(d_tie, w);
    if (c_tie <= 4) return c_tie == 1 ? wn.c[1] : c_tie == 2 ? wn.c[2] : c_tie == 3 ? wn.c[3] : wn.c[4];
    const uint32_t* row = bm + (d_tie - 1) * nwords;
    const uint16_t* jrow = jump + (d_tie - 1) * nwords;
    uint32_t big = wn.big, t = 0;
    while (big) {
      const int bit = __ffs(big) - 1;
      big &= big - 1;
      const int j = (w << 5) + bit;
      if (next_set(row, jrow, j) - j == c_tie) t |= 1u << bit;
    }
    return t;
  };
  if (listed) {
    for (uint32_t e = tid; e < big_total; e += NT) {
      const int c = (int)big_c[e], d = (int)(big_dj[e] >> 16);
      if (key_of(c, d) > tstar) keep(d, (int)(big_dj[e] & 0xFFFFu), c);
    }
  }
  // the light nodes can only be wanted when the heavy ones do not fill the tree
  if (!listed || tstar < key_of(5, kMaxM))
  for (int item = tid; item < items; item += NT) {
    const int d = item / nw + 1, w = item - (d - 1) * nw;
    const WordNodes wn = word_nodes(d, w);
#pragma unroll
    for (int c = 1; c <= 4; ++c) {
      if (key_of(c, d) > tstar && wn.c[c]) keep_bits(d, w, c, wn.c[c], (uint32_t)__popc(wn.c[c]));
    }
    const uint32_t* row = bm + (d - 1) * nwords;
    const uint16_t* jrow = jump + (d - 1) * nwords;
    uint32_t big = listed ? 0u : wn.big;
    while (big) {
      const int j = (w << 5) + __ffs(big) - 1;
      big &= big - 1;
      const int c = next_set(row, jrow, j) - j;
      if (key_of(c, d) > tstar) keep(d, j, c);
    }
  }
  if (r_tie > 0) {   // block-uniform
    for (int w = tid; w < nw; w += NT) tiecnt[w] = (uint16_t)__popc(tie_bits(w));
    __syncthreads();
    if (warp == 0) {                               // exclusive prefix sum over the words, in place
      uint32_t carry = 0;
      for (int c0 = 0; c0 < nw; c0 += 32) {
        const int w = c0 + lane;
        const uint32_t v = w < nw ? tiecnt[w] : 0u;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t u = __shfl_up_sync(kFull, incl, o);
          if (lane >= o) incl += u;
        }
        if (w < nw) tiecnt[w] = (uint16_t)min(carry + incl - v, 0xFFFFu);
        carry += __shfl_sync(kFull, incl, 31);
      }
    }
    __syncthreads();
    for (int w = tid; w < nw; w += NT) {
      uint32_t rank = tiecnt[w];
      if (rank >= r_tie) continue;
      const uint32_t t = tie_bits(w);
      const uint32_t take = min((uint32_t)__popc(t), r_tie - rank);
      if (take) keep_bits(d_tie, w, c_tie, t, take);
    }
  }
  __syncthreads();
  const int nn = (int)min(s.nsel, (uint32_t)N);
  if (s.nsel > (uint32_t)N && tid == 0) atomicOr(&s.err, REST_CTX_INTERNAL);

  // ---- phase 4: breadth-first order, parents, masks, tokens ---------------------------------
  // rank of a kept node = kept nodes with a smaller (depth, row); four threads share a node
  for (int idx0 = 0; idx0 < 4 * nn; idx0 += NT) {      // the same trip count for every thread
    const int idx = idx0 + tid, i = idx >> 2, q = idx & 3;
    uint32_t me = 0;
    int rank = 0;
    if (i < nn) {
      me = s.sel[i];
      for (int k = q; k < nn; k += 4) rank += (s.sel[k] < me);     // the four read neighbouring words
    }
    rank += __shfl_xor_sync(kFull, rank, 1);
    rank += __shfl_xor_sync(kFull, rank, 2);
    if (i < nn && q == 0) {
      s.sorted[rank] = me;
      s.sortedcnt[rank] = s.selcnt[i];
    }
  }
  __syncthreads();
  for (int i = tid; i < nn; i += NT) {
    const uint32_t me = s.sorted[i];
    const int d = (int)(me >> 16), j = (int)(me & 0xFFFFu);
    int par = -1;
    if (d > 1) {
      // the parent is the node of depth d - 1 whose rows include row j: the kept set is closed
      // under ancestors, so it is the last kept node (in breadth-first order) that starts at or
      // before row j at depth d - 1
      const uint32_t pmax = ((uint32_t)(d - 1) << 16) | (uint32_t)j;
      int l = 0, r = nn;                   // first kept node whose key exceeds pmax
      while (l < r) {
        const int mid = (l + r) >> 1;
        if (s.sorted[mid] <= pmax) l = mid + 1; else r = mid;
      }
      par = l - 1;
      bool ok = par >= 0 && (int)(s.sorted[par] >> 16) == d - 1;
      if (ok) {                            // and no node of that depth may start between it and row j
        const int jp = (int)(s.sorted[par] & 0xFFFFu);
        ok = next_set(bm + (d - 2) * nwords, jump + (d - 2) * nwords, jp) > j;
      }
      if (!ok) { atomicOr(&s.err, REST_CTX_INTERNAL); par = -1; }
    }
    s.par[i] = par;
    int64_t p;
    if (j < pcache_rows) p = (int64_t)pcache[j];
    else if constexpr (PART == kFromRuns) p = (int64_t)a.order[(int64_t)b * a.kcap + j] * m;
    else p = (int64_t)__ldg(sa + sample_slot(lo, cnt, a.K, a.sample_mode, j));
    int64_t o = (int64_t)b * N + i;
    a.tokens[o] = __ldg(Trow + p + n_win + d - 1);
    a.parents[o] = par;
    a.depth[o] = d;
    a.pos_ids[o] = clen + d - 1;
    if (a.node_count) a.node_count[o] = (int32_t)s.sortedcnt[i];
  }
  __syncthreads();
  // ancestor masks, a thread per (node, mask word): walk up the parents, keep the bits of its word
  for (int idx = tid; idx < nn * Wm; idx += NT) {
    const int i = idx / Wm, wq = idx - i * Wm;
    uint32_t bits = 0;
    int k = i;
    for (int step = 0; step <= kMaxM && k >= 0; ++step) {
      if ((k >> 5) == wq) bits |= 1u << (k & 31);
      k = s.par[k];
    }
    a.mask[((int64_t)b * N + i) * Wm + wq] = bits;
  }
  __syncthreads();
  if (s.err != 0) {
    // an inconsistency met while the tree was being written: the caller gets the empty tree
    // that every other reported problem gives, not a half-built one
    write_defaults();
    if (tid == 0) report_empty();
    return;
  }
  if (tid == 0) {
    a.status[b] = 0;
    a.n_nodes[b] = nn;
    if (a.match_n) a.match_n[b] = n_win;
    if (a.match_range) { a.match_range[2 * b] = lo; a.match_range[2 * b + 1] = hi; }
  }
}

template <typename SaT, bool TP, int NT, int PART>
__global__ void __launch_bounds__(NT, 1024 / NT)
rest_draft_kernel(DraftArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if constexpr (PART != kWholeShare) {
    draft_block<SaT, TP, NT, PART>(a, smem_raw);
  } else {
    // blocks beyond the contexts only help
    constexpr int NW = NT / 32;
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool has_context = (int)blockIdx.x < a.B;
    if (has_context) {
      if (tid == 0) atomicAdd(a.sh_hdr, 1);
      draft_block<SaT, TP, NT, PART>(a, smem_raw);
    } else if (tid == 0) {
      s.counted = 1;
    }
    __syncthreads();
    if (tid == 0 && !s.counted) atomicAdd(a.sh_hdr + 1, 1);     // left before its gather: nothing to offer
    // ---- help: while contexts may still offer rows, work on what is offered ---------------------
    long long* slot_base = reinterpret_cast<long long*>(smem_raw + sizeof(Smem));
    int* slot_len = reinterpret_cast<int*>(slot_base + NW * 34 + a.pcache_rows);
    const int32_t** my_sb = reinterpret_cast<const int32_t**>(slot_base + warp * 34);
    int* my_sl = slot_len + warp * 34;
    const int B = a.B;
    int polls = 0;
    for (;;) {
      if (warp == 0) {
        // anything offered?  (all warps then look for themselves)
        bool open = false;
        for (int k = 0; k < B; k += 32) {
          const int bb = k + lane;
          const int st = bb < B ? *reinterpret_cast<volatile int32_t*>(a.sh_ready + bb) : 0;
          open = open || __any_sync(kFull, st == 1);
        }
        int verdict = open ? 1 : 0;
        if (!open) {
          // Leave when nothing can come any more, or when contexts of this launch still wait
          // for an SM (a block that only helps gives them time to start), or after a while
          const int started = *reinterpret_cast<volatile int32_t*>(a.sh_hdr);
          const int past = *reinterpret_cast<volatile int32_t*>(a.sh_hdr + 1);
          if (past >= B || (started < B && has_context) || ++polls > kHelperPolls) verdict = -1;
          else __nanosleep(500);
        }
        if (lane == 0) s.help_b = verdict;
      }
      __syncthreads();
      const int verdict = s.help_b;
      __syncthreads();
      if (verdict < 0) break;
      if (verdict > 0) share_help_pass<SaT, NT>(a, s, my_sb, my_sl, (int)blockIdx.x % B, false);
    }
  }
}

// Dynamic shared memory of a block of `threads` threads that builds trees from up to K rows of
// m tokens (the search-only launch needs sizeof(Smem) alone).
size_t draft_smem_bytes(int K, int m, int threads, int* kcap_out, int* nwords_out, int* pcache_out,
                        int* bigcap_out) {
  const int kcap = (K + 31) / 32 * 32;
  const int nwords = kcap / 32 + 1;
  const int warps = threads / 32;
  const int pcache_rows = kcap < kPositionCacheRows ? kcap : kPositionCacheRows;
  if (kcap_out) *kcap_out = kcap;
  if (nwords_out) *nwords_out = nwords;
  if (pcache_out) *pcache_out = pcache_rows;
  // every fifth row at most starts a node of weight >= 5 at a depth
  const int bigcap = kcap < kBigListCap ? kcap : kBigListCap;
  if (bigcap_out) *bigcap_out = bigcap;
  size_t bytes = sizeof(Smem);
  bytes += (size_t)warps * 34 * 8;                         // slots: start positions
  bytes += (size_t)pcache_rows * 8;                        // suffix positions of the first rows
  bytes += (size_t)warps * 34 * 4;                         // slots: lengths
  bytes += (size_t)m * nwords * 4;                         // node-start bitmaps
  bytes += (size_t)m * nwords * 2;                         // jump tables
  bytes += (size_t)nwords * 2;                             // tie counts
  bytes += (size_t)bigcap * 6;                             // list of the heavy nodes
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
  if (wants_batched(prm->search_path, B, true, &batched) != REST_OK) return 0;
  if (batched) return split_workspace_bytes(B);
  // the one-launch form: scratch for shared gathering, where it can help
  if (!wants_share(prm->K, B) || prm->m < 1 || prm->m > REST_MAX_M || prm->K > REST_MAX_K) return 0;
  int nwords = 0;
  draft_smem_bytes(prm->K, prm->m, kThreads, nullptr, &nwords, nullptr, nullptr);
  return share_layout(B, prm->m, nwords).bytes;
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
  a.T = ds->v.tokens; a.sa = ds->v.sa; a.n_tokens = ds->v.n_tokens; a.n_sa = ds->v.n_sa; a.vocab = ds->v.vocab;
  a.n_max = prm->n_max; a.n_min = prm->n_min; a.K = prm->K; a.m = prm->m; a.N = prm->N;
  a.sample_mode = sample_mode;
  a.ctx = d_ctx; a.ctx_stride = ctx_stride; a.ctx_len = d_ctx_len;
  a.tokens = d_tokens; a.parents = d_parents; a.depth = d_depth; a.pos_ids = d_pos_ids;
  a.mask = d_mask; a.n_nodes = d_n_nodes; a.match_n = d_match_n; a.match_range = d_match_range;
  a.node_count = d_node_count; a.status = d_status;
  a.idx = ds->v.idx;
  auto smem_for = [&](int K, int threads) { return draft_smem_bytes(K, prm->m, threads, &a.kcap, &a.nwords, &a.pcache_rows, &a.bigcap); };
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool with_scratch = d_ws && ws_bytes >= split_workspace_bytes(B);
  bool batched = false;
  if (rest_status rc = wants_batched(search, B, with_scratch, &batched); rc != REST_OK) return rc;
  const bool narrow = ds->v.sa_bytes == 4;
  a.list = nullptr; a.list_count = nullptr; a.B = B; a.which = 0; a.light_rows = 0;
  a.kcap = 0; a.nwords = 0; a.pcache_rows = 0; a.bigcap = 0;
  a.sh_hdr = nullptr; a.sh_ready = nullptr; a.sh_desc = nullptr; a.sh_trunc = nullptr; a.sh_bm = nullptr; a.share_rows = 0;
  auto launch = [&](auto kern, int slot, int threads, int blocks, size_t bytes) -> rest_status {
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(kern),
                                            rest::kSmemSlotDraft + slot + (narrow ? 0 : 1), bytes));
    kern<<<blocks, threads, bytes, st>>>(a);
    rest::count_launch();
    REST_CUDA_TRY(cudaGetLastError());
    return REST_OK;
  };
  // candidate lists this long get 1024-thread blocks on every path
  const bool big = (size_t)prm->K * prm->m >= kBigRowsTimesM;
  if (!batched) {
    // a call with at most one context per SM lasts as long as its slowest context: give each
    // context the whole SM (not the single context: its typical candidate list is short and
    // the larger block only adds barrier time)
    const int sms = rest::sm_count();
    const bool wide_block = big || (B > 1 && B <= sms);
    const int threads = wide_block ? kBigThreads : kThreads;
    const size_t smem = smem_for(prm->K, threads);
    // With the caller's scratch, contexts with long candidate lists share their gather with
    // the blocks that are idle: those of finished contexts and, when the call has fewer contexts
    // than the GPU has SMs, blocks launched for nothing else (one per SM left over, so that
    // every block of the launch is resident at once).
    const ShareLayout lay = share_layout(B, prm->m, a.nwords);
    const bool share = d_ws && ws_bytes >= lay.bytes && reinterpret_cast<uintptr_t>(d_ws) % 16 == 0 &&
                       wants_share(prm->K, B);
    if (share) {
      unsigned char* ws = static_cast<unsigned char*>(d_ws);
      a.sh_hdr = reinterpret_cast<int32_t*>(ws);
      a.sh_ready = reinterpret_cast<int32_t*>(ws + lay.ready);
      a.sh_desc = reinterpret_cast<ShareDesc*>(ws + lay.desc);
      a.sh_trunc = reinterpret_cast<uint32_t*>(ws + lay.trunc);
      a.sh_bm = reinterpret_cast<uint32_t*>(ws + lay.bm);
      a.share_rows = kShareRows;
      REST_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.zeroed_bytes, st));
      const int blocks = B < sms ? sms : B;
      if (wide_block)
        return narrow ? launch(rest_draft_kernel<int32_t, false, kBigThreads, kWholeShare>, 18, kBigThreads, blocks, smem)
                      : launch(rest_draft_kernel<int64_t, false, kBigThreads, kWholeShare>, 18, kBigThreads, blocks, smem);
      return narrow ? launch(rest_draft_kernel<int32_t, false, kThreads, kWholeShare>, 16, kThreads, blocks, smem)
                    : launch(rest_draft_kernel<int64_t, false, kThreads, kWholeShare>, 16, kThreads, blocks, smem);
    }
    if (wide_block)
      return narrow ? launch(rest_draft_kernel<int32_t, false, kBigThreads, kWhole>, 10, kBigThreads, B, smem)
                    : launch(rest_draft_kernel<int64_t, false, kBigThreads, kWhole>, 10, kBigThreads, B, smem);
    return narrow ? launch(rest_draft_kernel<int32_t, false, kThreads, kWhole>, 0, kThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, false, kThreads, kWhole>, 0, kThreads, B, smem);
  }
  if (!with_scratch) {
    // no scratch for the context lists: search and build in one launch
    const size_t smem = smem_for(prm->K, kTpThreads);
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
  const size_t smem_light = smem_for(a.light_rows, kLightThreads);
  a.which = 0;
  rc = narrow ? launch(rest_draft_kernel<int32_t, true, kLightThreads, kBuild>, 6, kLightThreads, B, smem_light)
              : launch(rest_draft_kernel<int64_t, true, kLightThreads, kBuild>, 6, kLightThreads, B, smem_light);
  if (rc != REST_OK) return rc;
  if (prm->K > a.light_rows) {
    a.which = 1;
    if (big) {
      const size_t smem = smem_for(prm->K, kBigThreads);
      rc = narrow ? launch(rest_draft_kernel<int32_t, true, kBigThreads, kBuild>, 12, kBigThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, true, kBigThreads, kBuild>, 12, kBigThreads, B, smem);
    } else {
      const size_t smem = smem_for(prm->K, kThreads);
      rc = narrow ? launch(rest_draft_kernel<int32_t, true, kThreads, kBuild>, 8, kThreads, B, smem)
                  : launch(rest_draft_kernel<int64_t, true, kThreads, kBuild>, 8, kThreads, B, smem);
    }
  }
  return rc;
}

// ---------------------------------------------------------------------------------------
// The draft in pieces, for a datastore that is spread over several GPUs: every GPU searches
// its own shard (rest_retrieve), the shards agree on the winning suffix length and on how many
// candidates each contributes (a few collectives, the caller's business), every GPU reads its
// share of the candidate rows (rest_gather_rows), the rows travel, and the tree is built from
// the runs of all shards (rest_draft_from_runs).
// ---------------------------------------------------------------------------------------
namespace {

// One block per context: candidate j < take[b] of the matched range is slot lo + j when the
// whole range is taken, else lo + floor(j * cnt / take[b]); its up to m tokens and its length.
template <typename SaT>
__global__ void __launch_bounds__(256)
gather_rows_kernel(const int32_t* __restrict__ T, const SaT* __restrict__ sa, int64_t n_tokens, int64_t n_sa,
                   int m, int sample_mode, const int32_t* __restrict__ match_n,
                   const int64_t* __restrict__ match_range, const int32_t* __restrict__ take, int Kr,
                   int32_t* __restrict__ rows, int32_t* __restrict__ row_len, int32_t* __restrict__ status) {
  const int b = blockIdx.x;
  const int n = match_n[b];
  int64_t lo = match_range[2 * b], hi = match_range[2 * b + 1];
  lo = lo < 0 ? 0 : (lo > n_sa ? n_sa : lo);
  hi = hi < lo ? lo : (hi > n_sa ? n_sa : hi);
  const int64_t cnt = hi - lo;
  int k = take[b];
  k = k < 0 ? 0 : (k > Kr ? Kr : k);
  if ((int64_t)k > cnt) k = (int)cnt;
  if (n <= 0) k = 0;
  bool bad = false;
  for (int j = threadIdx.x; j < Kr; j += blockDim.x) {
    int32_t* out = rows + ((int64_t)b * Kr + j) * m;
    int len = 0;
    if (j < k) {
      const int64_t slot = sample_slot(lo, cnt, k, sample_mode, j);
      const int64_t p = (int64_t)__ldg(sa + slot);
      if (p < 0 || p >= n_tokens) {
        bad = true;
      } else {
        const int64_t rem = n_tokens - (p + n);
        len = (int)(rem < 0 ? 0 : (rem > m ? m : rem));
        for (int d = 0; d < len; ++d) out[d] = __ldg(T + p + n + d);
      }
    }
    for (int d = len; d < m; ++d) out[d] = 0;
    row_len[(int64_t)b * Kr + j] = len;
  }
  if (bad) atomicOr(status + b, REST_CTX_BAD_DATASTORE);
}

}  // namespace

extern "C" rest_status rest_retrieve(const rest_datastore* ds, const rest_draft_params* prm,
                                     const int32_t* d_ctx, int64_t ctx_stride, const int32_t* d_ctx_len,
                                     int32_t B, int32_t* d_match_n, int64_t* d_match_range,
                                     int32_t* d_status, void* stream) {
  if (!ds || !prm || B < 0) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_ctx || !d_ctx_len || !d_match_n || !d_match_range || !d_status || ctx_stride < 0) return REST_INVALID_ARG;
  if (prm->n_min < 1 || prm->n_max < prm->n_min) return REST_INVALID_ARG;
  if (prm->n_max > REST_MAX_SUFFIX || prm->n_max - prm->n_min + 1 > kWarps) return REST_UNSUPPORTED;
  DraftArgs a = {};
  a.T = ds->v.tokens; a.sa = ds->v.sa; a.n_tokens = ds->v.n_tokens; a.n_sa = ds->v.n_sa; a.vocab = ds->v.vocab;
  a.idx = ds->v.idx;
  a.n_max = prm->n_max; a.n_min = prm->n_min; a.K = 1; a.m = 1; a.N = 1; a.sample_mode = 0;
  a.ctx = d_ctx; a.ctx_stride = ctx_stride; a.ctx_len = d_ctx_len;
  a.match_n = d_match_n; a.match_range = d_match_range; a.status = d_status; a.B = B;
  const bool narrow = ds->v.sa_bytes == 4;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (narrow) rest_draft_kernel<int32_t, false, kThreads, kRetrieve><<<B, kThreads, sizeof(Smem), st>>>(a);
  else rest_draft_kernel<int64_t, false, kThreads, kRetrieve><<<B, kThreads, sizeof(Smem), st>>>(a);
  rest::count_launch();
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}

extern "C" rest_status rest_gather_rows(const rest_datastore* ds, const rest_draft_params* prm,
                                        const int32_t* d_match_n, const int64_t* d_match_range,
                                        const int32_t* d_take, int32_t B, int32_t Kr, int32_t* d_rows,
                                        int32_t* d_row_len, int32_t* d_status, void* stream) {
  if (!ds || !prm || B < 0 || Kr < 1) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_match_n || !d_match_range || !d_take || !d_rows || !d_row_len || !d_status) return REST_INVALID_ARG;
  if (prm->m < 1) return REST_INVALID_ARG;
  if (prm->m > REST_MAX_M || Kr > REST_MAX_K) return REST_UNSUPPORTED;
  if (prm->sample_mode != REST_SAMPLE_STRIDED && prm->sample_mode != REST_SAMPLE_FIRST_K) return REST_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (ds->v.sa_bytes == 4)
    gather_rows_kernel<int32_t><<<B, 256, 0, st>>>(ds->v.tokens, static_cast<const int32_t*>(ds->v.sa),
                                                   ds->v.n_tokens, ds->v.n_sa, prm->m, prm->sample_mode, d_match_n,
                                                   d_match_range, d_take, Kr, d_rows, d_row_len, d_status);
  else
    gather_rows_kernel<int64_t><<<B, 256, 0, st>>>(ds->v.tokens, static_cast<const int64_t*>(ds->v.sa),
                                                   ds->v.n_tokens, ds->v.n_sa, prm->m, prm->sample_mode, d_match_n,
                                                   d_match_range, d_take, Kr, d_rows, d_row_len, d_status);
  rest::count_launch();
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}

extern "C" size_t rest_draft_from_runs_workspace_bytes(int32_t B, int32_t R, int32_t Kr) {
  if (B <= 0 || R <= 0 || Kr <= 0) return 0;
  const size_t kcap = ((size_t)R * Kr + 31) / 32 * 32;
  return (size_t)B * kcap * sizeof(uint32_t);
}

extern "C" rest_status rest_draft_from_runs(const rest_draft_params* prm, const int32_t* d_rows,
                                            const int32_t* d_row_len, const int32_t* d_run_rows, int32_t R,
                                            int32_t Kr, const int32_t* d_ctx_len, int32_t B,
                                            int32_t* d_tokens, int32_t* d_parents, int32_t* d_depth,
                                            int32_t* d_pos_ids, uint32_t* d_mask, int32_t* d_n_nodes,
                                            int32_t* d_node_count, int32_t* d_status, void* d_ws,
                                            size_t ws_bytes, void* stream) {
  if (!prm || B < 0 || R < 1 || Kr < 1) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_rows || !d_row_len || !d_run_rows || !d_ctx_len || !d_tokens || !d_parents || !d_depth ||
      !d_pos_ids || !d_mask || !d_n_nodes || !d_status)
    return REST_INVALID_ARG;
  if (prm->m < 1 || prm->N < 1) return REST_INVALID_ARG;
  if (prm->m > REST_MAX_M || prm->N > REST_MAX_N || (int64_t)R * Kr > REST_MAX_K) return REST_UNSUPPORTED;
  const size_t need = rest_draft_from_runs_workspace_bytes(B, R, Kr);
  if (!d_ws) return REST_INVALID_ARG;
  if (ws_bytes < need) return REST_WORKSPACE_TOO_SMALL;
  DraftArgs a = {};
  a.T = d_rows; a.row_len = d_row_len; a.run_rows = d_run_rows; a.R = R; a.Kr = Kr;
  a.order = static_cast<uint32_t*>(d_ws);
  a.n_tokens = (int64_t)B * R * Kr * prm->m; a.n_sa = a.n_tokens; a.vocab = 0x7FFFFFFFu;
  a.n_max = 0; a.n_min = 0; a.K = R * Kr; a.m = prm->m; a.N = prm->N; a.sample_mode = 0;
  a.ctx_len = d_ctx_len;
  a.tokens = d_tokens; a.parents = d_parents; a.depth = d_depth; a.pos_ids = d_pos_ids; a.mask = d_mask;
  a.n_nodes = d_n_nodes; a.node_count = d_node_count; a.status = d_status; a.B = B;
  const bool big = (size_t)a.K * prm->m >= kBigRowsTimesM;
  const int threads = big ? kBigThreads : kThreads;
  const size_t smem = draft_smem_bytes(a.K, prm->m, threads, &a.kcap, &a.nwords, &a.pcache_rows, &a.bigcap);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (big) {
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(rest_draft_kernel<int32_t, false, kBigThreads, kFromRuns>),
                                            rest::kSmemSlotDraft + 15, smem));
    rest_draft_kernel<int32_t, false, kBigThreads, kFromRuns><<<B, kBigThreads, smem, st>>>(a);
  } else {
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(rest_draft_kernel<int32_t, false, kThreads, kFromRuns>),
                                            rest::kSmemSlotDraft + 14, smem));
    rest_draft_kernel<int32_t, false, kThreads, kFromRuns><<<B, kThreads, smem, st>>>(a);
  }
  rest::count_launch();
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}
