// rest_tree_attention: masked attention of the N draft positions over the prefix KV cache
// and over their own ancestors (Sec. 3.2 "Draft verification").
//
// Split-KV flash-decode layout on the 5th-generation tensor cores.  One thread block per
// (context, head, 64-row block of the draft rows, key split) streams 64-key K/V tiles:
// S = Q K^T and O += P V are tcgen05.mma with the accumulators in TMEM, the operand tiles
// arrive by TMA, and the tree mask / base-2 online softmax runs in registers in between.
//
// M = 64 rather than 128 because an M = 64 accumulator spreads its rows over all four TMEM
// lane quadrants (16 rows each), so every softmax warp - and every warp scheduler - gets an
// equal share.  Every 64-row block of the N draft rows gets its own thread blocks (grid
// index: row block fastest after the split, so the blocks of one (context, head) stream the
// same K/V tiles at the same time and the second reader hits L2).
//
// Q ([64 x 128]), the K/V tiles ([64 x 128]) and P ([64 x 64]) sit in shared memory in the
// tensor core's canonical 128-byte-swizzled layout (8-row groups of 1024 B, the two
// 64-element halves of the head dimension side by side), so a K tile is a K-major B operand
// and the very same bytes of a V tile are an MN-major B operand: no transpose anywhere.
// Per 64-key tile:
//   8 tcgen05.mma (M=64, N=64, K=16)   ->  S in TMEM columns [0, 64) or [64, 128)
//   each softmax warp reads its 16 rows with the 16x256b pattern (a row is shared by a quad),
//   applies scale / tree mask / online softmax, and writes P (bf16) into shared memory
//   4 tcgen05.mma (M=64, N=128, K=16)  ->  P V in TMEM columns [128, 256)
//   each warp folds its rows of P V into fp32 register accumulators with the usual rescale.
//
// The splits of one (context, head, row block) form a thread-block cluster (up to 8 blocks).
// Every block stages its un-normalised partial rows in its own shared memory and sends each
// owner its slice with one bulk shared-to-shared copy that completes on the owner's
// mbarrier; the owner reduces locally and writes bf16 output.  Only when more than 8 splits
// are needed do the cluster-merged partials go to the caller's workspace for a second, small
// merge kernel.
#include <atomic>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kD = REST_HEAD_DIM;     // 128
constexpr int kBN = 64;               // keys per tile
constexpr int kOStride = kD + 4;      // floats per row of a staged partial: 128 O + m, l (+2 pad)
constexpr int kMaxCluster = 8;
constexpr int kRowBytes = kD * 2;     // 256
constexpr int kTileBytes = kBN * kRowBytes;   // 16 KB
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttnArgs {
  const __nv_bfloat16 *q, *k, *v;
  __nv_bfloat16* out;
  float* lse;
  const int32_t* kv_len;
  const uint32_t* mask;
  float* ws_o;      // [B,H,Sp,N,128] fp32 partial numerators (Sp = clusters per (b,h))
  float* ws_ml;     // [B,H,Sp,N,2]   running max (base-2 units) and sum
  int64_t q_b, q_n, q_h, kv_b, kv_h, kv_l, o_b, o_n, o_h;
  int B, H, group, N, Wm;
  int S;            // key splits per (context, head) = C * Sp
  int NBLK;         // 128-row query blocks per (context, head) in the wide kernel (else 1)
  int unit0;        // first unit (context, head, row block) of this launch
  int pack;         // query heads per block in the wide kernel: 2 when N = 64 and heads share KV
  int q_slot[3], kv_slot[3];   // tensor-map coordinate index (1..3) of rows, head, batch
  int C;            // blocks per cluster
  int Sp;           // clusters per (context, head); > 1 needs the merge kernel
  float scale_log2;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr int kTcStages = 2;                            // K and V ring depth
constexpr int kQBlockBytes = 64 * kRowBytes;            // 16 KB: 64 rows x 128 dims
constexpr int kPBlockBytes = 64 * 128;                  //  8 KB: 64 rows x 64 keys
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColO = 128;      // S double-buffered in [0,64) and [64,128); P V in [128,256)
constexpr long long kWaitCycles = 400000000ll;          // ~0.2 s: give up, flag, clean up

// Shared memory: operand tiles (Q blocks, K ring, V ring, P blocks), later reused by the split
// merge, which stages 64 NB partial rows and receives up to 64 NB + 8 rows of kOStride floats;
// the mbarriers and the TMEM slot sit behind whichever is larger.  (NB = 64-row blocks per
// thread block; the kernel uses NB = 1, which keeps two blocks resident per SM.)
__host__ __device__ constexpr int tc_operand_bytes(int NB) { return NB * kQBlockBytes + 2 * kTcStages * kTileBytes + NB * kPBlockBytes; }
__host__ __device__ constexpr int tc_merge_bytes(int NB) { return (2 * 64 * NB + 8) * kOStride * 4; }
__host__ __device__ constexpr int tc_bar_offset(int NB) {
  return tc_operand_bytes(NB) > tc_merge_bytes(NB) ? tc_operand_bytes(NB) : tc_merge_bytes(NB);
}
// Tiles are dealt so that the first splits take the spare ones: the last split, which holds
// the masked tree tiles, never gets an extra tile.
__host__ __device__ inline int tc_tile_begin(int split, int ntiles, int S) {
  return (int)(((long long)split * ntiles + S - 1) / S);
}

__device__ unsigned int g_attn_error;                   // bit 0: wait gave up, bit 1: smem misaligned

// shared-memory matrix descriptor: 128-byte swizzle, descriptor version 1
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major (0) or MN-major (1)
__device__ __forceinline__ constexpr uint32_t umma_idesc(int M, int N, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                         uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 16 TMEM lanes x 64 columns: r[4k..4k+3] = {row g: cols 8k+2t, 8k+2t+1; row g+8: same cols}
__device__ __forceinline__ void tmem_ld_16x64(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Bounded wait on an mbarrier phase; false when the time limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  const long long start = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (clock64() - start > kWaitCycles) return false;
  }
}

// =======================================================================================
// The kernel is warp-specialised: three kinds of work run in their own warps and talk through
// mbarriers only; there is no block-wide barrier inside the loop:
//   warp 4, one thread: TMA producer.  K and V tiles (and Q once) arrive as 64 x 64 boxes of
//           a 4-D tensor map with 128-byte swizzle, which is exactly the operand layout; rows
//           past the tensor's extent are zero-filled by the copy engine.  A slot is refilled
//           as soon as the MMA that read it has completed (tcgen05.commit on its "free" barrier).
//   warp 5, one thread: MMA issuer.  Q K(t+2)^T is issued right after P V(t), so the tensor
//           core always has the next S tile ready while the softmax warps work on this one.
//   warps 0..3: softmax.  Wait for S(t), read it from TMEM, scale / mask / online softmax, fold
//           P V(t-1) into the register accumulators, store P(t), signal the MMA warp.
// Every wait is bounded; a wait that gives up raises a block-wide abort word that every other
// wait polls, so all roles leave their loops and the block still frees its TMEM; the host
// reads the failure through rest_device_error_flags.
// =======================================================================================
constexpr int kWsThreads = 192;
constexpr int kWsBarBytes = 192;
// barrier slots (8 bytes each) behind the operand tiles
enum {
  kBarKFull = 0, kBarVFull = 16, kBarSFull = 32, kBarOFull = 48, kBarKFree = 56, kBarVFree = 72,
  kBarPFull = 88, kBarQFull = 96, kBarMerge = 104, kBarTmemSlot = 112, kBarAbort = 116
};
__host__ __device__ constexpr int ws_smem_bytes() { return tc_bar_offset(1) + kWsBarBytes; }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait that also gives up when another thread of the block has raised the abort word.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, volatile uint32_t* abort_word) {
  const long long start = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (*abort_word != 0u) return false;
    if (clock64() - start > kWaitCycles) { *abort_word = 1u; return false; }
  }
}
// one 64 x 64 bf16 box (8 KB) of a 4-D tensor map -> shared memory, completion on an mbarrier
// (row, head, batch) sit at tensor-map coordinates slot[0], slot[1], slot[2] (each 1..3): the map
// orders its outer dimensions by increasing stride, whatever the caller's layout is.
__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, int c0, int row, int head,
                                             int batch, const int (&slot)[3], uint32_t bar) {
  const int c1 = slot[0] == 1 ? row : slot[1] == 1 ? head : batch;
  const int c2 = slot[0] == 2 ? row : slot[1] == 2 ? head : batch;
  const int c3 = slot[0] == 3 ? row : slot[1] == 3 ? head : batch;
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__global__ void __launch_bounds__(kWsThreads, 2)
tree_attention_ws_kernel(AttnArgs a, const __grid_constant__ CUtensorMap tm_q,
                         const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v) {
  constexpr int NB = 1;
  extern __shared__ __align__(1024) unsigned char smem[];
  const int N = a.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool is_softmax = warp < 4;
  const int g = lane >> 2, t4 = lane & 3;
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase;
  const uint32_t sK = sQ + kQBlockBytes;
  const uint32_t sV = sK + kTcStages * kTileBytes;
  const uint32_t sP = sV + kTcStages * kTileBytes;
  const uint32_t bars = sbase + tc_bar_offset(1);
  const uint32_t bar_m = bars + kBarMerge;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + tc_bar_offset(1) + kBarTmemSlot);
  volatile uint32_t* abort_word = reinterpret_cast<volatile uint32_t*>(smem + tc_bar_offset(1) + kBarAbort);

  int bid = blockIdx.x;
  const int split = bid % a.S; bid = bid / a.S + a.unit0;
  const int h = bid % a.H;
  const int b = bid / a.H;
  const int hk = h / a.group;
  constexpr int row0 = 0;                            // this kernel serves N <= 64: one row block
  const int Nl = N;                                  // its number of real rows

  // Programmatic dependent launch: the next kernel in the stream may start its own set-up now;
  // this kernel touches no global memory until the one before it has fully completed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if ((sbase & 1023u) != 0) {   // the swizzled operand layout needs a 1024-byte aligned base
    if (tid == 0) atomicOr(&g_attn_error, 2u);
    return;                     // uniform over the grid: every block sees the same offset
  }

  if (tid == 0) {
    mbar_init(bars + kBarKFull, 1); mbar_init(bars + kBarKFull + 8, 1);
    mbar_init(bars + kBarVFull, 1); mbar_init(bars + kBarVFull + 8, 1);
    mbar_init(bars + kBarSFull, 1); mbar_init(bars + kBarSFull + 8, 1);
    mbar_init(bars + kBarOFull, 1);
    mbar_init(bars + kBarKFree, 1); mbar_init(bars + kBarKFree + 8, 1);
    mbar_init(bars + kBarVFree, 1); mbar_init(bars + kBarVFree + 8, 1);
    mbar_init(bars + kBarPFull, 4);            // one arrival per softmax warp
    mbar_init(bars + kBarQFull, 1);
    mbar_init(bar_m, 1);
    *abort_word = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (a.S > 1) {   // merge: this block will receive its rows of every peer's partial
      const int Rm = (Nl + a.C - 1) / a.C;
      const int mine = max(0, min(Rm, Nl - (split % a.C) * Rm));
      mbar_expect_tx(bar_m, (uint32_t)(a.C * mine * kOStride * 4));
    }
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // everything above is independent of the inputs; from here on global memory is read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int L = a.kv_len[b];
  const int total = L + N;
  const int ntiles = (total + kBN - 1) / kBN;
  const int t0 = tc_tile_begin(split, ntiles, a.S);
  const int t1 = tc_tile_begin(split + 1, ntiles, a.S);
  const int nt = t1 - t0;

  // rows of this thread (softmax warps): rows 16 warp + g and + 8; mask row as two 64-bit halves
  unsigned long long mlo[NB][2], mhi[NB][2];
  float o[NB][16][4];
  float m_run[NB][2], l_run[NB][2], alpha[NB][2];
#pragma unroll
  for (int rb = 0; rb < NB; ++rb) {
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int row = (warp & 3) * 16 + g + 8 * hh;
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (is_softmax && row < Nl) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (i < a.Wm) w[i] = a.mask[((int64_t)b * N + row0 + row) * a.Wm + i];
      }
      mlo[rb][hh] = (unsigned long long)w[0] | ((unsigned long long)w[1] << 32);
      mhi[rb][hh] = (unsigned long long)w[2] | ((unsigned long long)w[3] << 32);
      m_run[rb][hh] = -INFINITY; l_run[rb][hh] = 0.f; alpha[rb][hh] = 1.f;
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[rb][i][0] = o[rb][i][1] = o[rb][i][2] = o[rb][i][3] = 0.f; }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_warp = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      mbar_expect_tx(bars + kBarQFull, (uint32_t)kQBlockBytes);
      tma_load_box(sQ, &tm_q, 0, row0, h, b, a.q_slot, bars + kBarQFull);
      tma_load_box(sQ + 64 * 128, &tm_q, 64, row0, h, b, a.q_slot, bars + kBarQFull);
    }
    // K tiles by lane 0, V tiles by lane 1: a K slot frees as soon as its Q K^T has run, a V slot
    // only after the softmax and P V of its tile; one thread issuing both in turn would hold the
    // next K tile back behind the wait for a V slot.
    if (lane < 2) {
      const bool is_v = lane == 1;
      const uint32_t ring = is_v ? sV : sK;
      const CUtensorMap* map = is_v ? &tm_v : &tm_k;
      const uint32_t full = bars + (is_v ? kBarVFull : kBarKFull), free_ = bars + (is_v ? kBarVFree : kBarKFree);
      int issued = 0;
      for (int it = 0; it < nt; ++it) {
        const int slot = it & 1, key0 = (t0 + it) * kBN;
        const uint32_t free_parity = (uint32_t)(((it >> 1) + 1) & 1);
        if (it >= 2 && !mbar_wait_abortable(free_ + slot * 8, free_parity, abort_word)) break;
        mbar_expect_tx(full + slot * 8, (uint32_t)kTileBytes);
        tma_load_box(ring + slot * kTileBytes, map, 0, key0, hk, b, a.kv_slot, full + slot * 8);
        tma_load_box(ring + slot * kTileBytes + 64 * 128, map, 64, key0, hk, b, a.kv_slot, full + slot * 8);
        ++issued;
      }
      if (*abort_word != 0u) {
        // giving up: let the copies already in flight land before this block goes away
        if (!is_v) mbar_wait(bars + kBarQFull, 0u);
        for (int it = max(0, issued - 2); it < issued; ++it)
          mbar_wait(full + (it & 1) * 8, (uint32_t)((it >> 1) & 1));
      }
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc(64, kBN, 0);
      constexpr uint32_t idesc_o = umma_idesc(64, kD, 1);
      const uint64_t dq0 = umma_desc(sQ, 16, 1024);
      const uint64_t dk0 = umma_desc(sK, 16, 1024);
      const uint64_t dp0 = umma_desc(sP, 16, 1024);
      const uint64_t dv0 = umma_desc(sV, kBN * 128, 1024);
      bool ok = mbar_wait_abortable(bars + kBarQFull, 0u, abort_word);
      // S[it & 1] = Q K(t)^T.  The S buffer is free: its previous reader stored P(it - 2) only
      // after reading it, and P(it - 2) was waited for before this call.
      auto issue_qk = [&](int it) -> bool {
        const int slot = it & 1;
        if (!mbar_wait_abortable(bars + kBarKFull + slot * 8, (uint32_t)((it >> 1) & 1), abort_word)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t koff = (uint32_t)((ks >> 2) * (64 * 128) + (ks & 3) * 32);
          umma_f16(tmem_base + kColS + slot * 64, dq0 + (koff >> 4),
                   dk0 + ((slot * kTileBytes + koff) >> 4), idesc_s, ks > 0);
        }
        umma_commit(bars + kBarSFull + slot * 8);
        umma_commit(bars + kBarKFree + slot * 8);
        return true;
      };
      if (ok && nt > 0) ok = issue_qk(0);
      if (ok && nt > 1) ok = issue_qk(1);
      for (int it = 0; ok && it < nt; ++it) {
        const int slot = it & 1;
        // P(it) is in shared memory; its writers had folded P V(it - 1) before, so O is free
        if (!mbar_wait_abortable(bars + kBarPFull, (uint32_t)(it & 1), abort_word)) break;
        if (!mbar_wait_abortable(bars + kBarVFull + slot * 8, (uint32_t)((it >> 1) & 1), abort_word)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_f16(tmem_base + kColO, dp0 + ((kk * 32) >> 4),
                   dv0 + ((slot * kTileBytes + kk * 2048) >> 4), idesc_o, kk > 0);
        umma_commit(bars + kBarOFull);
        umma_commit(bars + kBarVFree + slot * 8);
        if (it + 2 < nt) ok = issue_qk(it + 2);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax warps
    auto fold_pv = [&]() {           // o = o * alpha + (P V of the previous tile)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t orr[32];
        tmem_ld_16x64(tmem_warp + kColO + hf * 64, orr);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          float* oo = o[0][hf * 8 + k];
          oo[0] = oo[0] * alpha[0][0] + __uint_as_float(orr[4 * k]);
          oo[1] = oo[1] * alpha[0][0] + __uint_as_float(orr[4 * k + 1]);
          oo[2] = oo[2] * alpha[0][1] + __uint_as_float(orr[4 * k + 2]);
          oo[3] = oo[3] * alpha[0][1] + __uint_as_float(orr[4 * k + 3]);
        }
      }
    };
    bool ok = true;
    for (int it = 0; ok && it < nt; ++it) {
      const int t = t0 + it;
      if (!mbar_wait_abortable(bars + kBarSFull + (it & 1) * 8, (uint32_t)((it >> 1) & 1), abort_word)) break;
      tc_fence_after();
      const int key0 = t * kBN;
      const bool need_mask = key0 + kBN > L;
      uint32_t pk[NB][16];
      float alpha_new[NB][2];
#pragma unroll
      for (int rb = 0; rb < NB; ++rb) {
        uint32_t sr[32];
        tmem_ld_16x64(tmem_warp + kColS + (it & 1) * 64, sr);
        tmem_wait_ld();
        float mx0 = -INFINITY, mx1 = -INFINITY;
        if (!need_mask) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float v0 = __uint_as_float(sr[4 * k]) * a.scale_log2, v1 = __uint_as_float(sr[4 * k + 1]) * a.scale_log2;
            const float v2 = __uint_as_float(sr[4 * k + 2]) * a.scale_log2, v3 = __uint_as_float(sr[4 * k + 3]) * a.scale_log2;
            sr[4 * k] = __float_as_uint(v0); sr[4 * k + 1] = __float_as_uint(v1);
            sr[4 * k + 2] = __float_as_uint(v2); sr[4 * k + 3] = __float_as_uint(v3);
            mx0 = fmaxf(mx0, fmaxf(v0, v1));
            mx1 = fmaxf(mx1, fmaxf(v2, v3));
          }
        } else {
          // 64-bit "key j of this tile is visible" masks of the thread's two rows: prefix keys,
          // then the row's tree bits moved to where key L sits in this tile
          unsigned long long am[2];
          const int off = L - key0;                // position of key L in this tile (may be < 0)
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            unsigned long long pre = off >= 64 ? ~0ull : (off <= 0 ? 0ull : ((1ull << off) - 1ull));
            unsigned long long tb;
            if (off >= 64) tb = 0ull;
            else if (off >= 0) tb = mlo[rb][hh] << off;
            else if (off > -64) tb = (mlo[rb][hh] >> (-off)) | (mhi[rb][hh] << (64 + off));
            else if (off > -128) tb = mhi[rb][hh] >> (-off - 64);
            else tb = 0ull;
            am[hh] = (pre | tb) >> (2 * t4);
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const bool ok = (am[e >> 1] >> (8 * k + (e & 1))) & 1ull;
              const float v = ok ? __uint_as_float(sr[4 * k + e]) * a.scale_log2 : -INFINITY;
              sr[4 * k + e] = __float_as_uint(v);
            }
            mx0 = fmaxf(mx0, fmaxf(__uint_as_float(sr[4 * k]), __uint_as_float(sr[4 * k + 1])));
            mx1 = fmaxf(mx1, fmaxf(__uint_as_float(sr[4 * k + 2]), __uint_as_float(sr[4 * k + 3])));
          }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
        const float mn0 = fmaxf(m_run[rb][0], mx0), mn1 = fmaxf(m_run[rb][1], mx1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        alpha_new[rb][0] = ex2(m_run[rb][0] - ms0);  // m = -inf gives 0
        alpha_new[rb][1] = ex2(m_run[rb][1] - ms1);
        m_run[rb][0] = mn0; m_run[rb][1] = mn1;
        float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float e0 = ex2(__uint_as_float(sr[4 * k]) - ms0), e1 = ex2(__uint_as_float(sr[4 * k + 1]) - ms0);
          const float e2 = ex2(__uint_as_float(sr[4 * k + 2]) - ms1), e3 = ex2(__uint_as_float(sr[4 * k + 3]) - ms1);
          ps0 += e0 + e1;
          ps1 += e2 + e3;
          pk[rb][2 * k] = pack_bf16(e0, e1);
          pk[rb][2 * k + 1] = pack_bf16(e2, e3);
        }
        l_run[rb][0] = l_run[rb][0] * alpha_new[rb][0] + ps0;
        l_run[rb][1] = l_run[rb][1] * alpha_new[rb][1] + ps1;
      }
      if (it > 0) {
        if (!mbar_wait_abortable(bars + kBarOFull, (uint32_t)((it - 1) & 1), abort_word)) break;
        tc_fence_after();
        fold_pv();
      }
      alpha[0][0] = alpha_new[0][0]; alpha[0][1] = alpha_new[0][1];
      if (key0 + kBN > total) {
        // Ragged last tile: rows of V past the last real key hold whatever the cache holds
        // there.  Their probabilities are zero, but 0 x NaN is NaN: clear them.
        if (!mbar_wait_abortable(bars + kBarVFull + (it & 1) * 8, (uint32_t)((it >> 1) & 1), abort_word)) break;
        const int first = total - key0;            // 0 < first < 64
        for (int c = tid; c < (kBN - first) * 16; c += 128) {
          const int row = first + (c >> 4), chunk = c & 15;
          const uint32_t dst = sV + (it & 1) * kTileBytes + (chunk >> 3) * (64 * 128) + (row >> 3) * 1024 +
                               (row & 7) * 128 + (((chunk & 7) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
        }
      }
      {
        // P (bf16) -> shared memory, K-major 128-byte-swizzled [64 rows x 64 keys]
        const int rr0 = warp * 16 + g, rr1 = rr0 + 8;
        const uint32_t p0 = sP + (rr0 >> 3) * 1024 + (rr0 & 7) * 128 + t4 * 4;
        const uint32_t p1 = sP + (rr1 >> 3) * 1024 + (rr1 & 7) * 128 + t4 * 4;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(p0 + ((k ^ (rr0 & 7)) << 4)), "r"(pk[0][2 * k]) : "memory");
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(p1 + ((k ^ (rr1 & 7)) << 4)), "r"(pk[0][2 * k + 1]) : "memory");
        }
      }
      fence_async_smem();                          // P (and cleared V rows) -> visible to the tensor core
      tc_fence_before();                           // this warp's TMEM reads are done
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + kBarPFull);
    }
    if (nt > 0 && *abort_word == 0u) {             // the last tile's P V
      if (mbar_wait_abortable(bars + kBarOFull, (uint32_t)((nt - 1) & 1), abort_word)) {
        tc_fence_after();
        fold_pv();
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_word != 0u && tid == 0) atomicOr(&g_attn_error, 1u);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }

#pragma unroll
  for (int rb = 0; rb < NB; ++rb) {
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[rb][hh] += __shfl_xor_sync(0xFFFFFFFFu, l_run[rb][hh], 1);
      l_run[rb][hh] += __shfl_xor_sync(0xFFFFFFFFu, l_run[rb][hh], 2);
    }
  }

  if (a.S == 1) {
#pragma unroll
    for (int rb = 0; rb < NB; ++rb) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int row = rb * 64 + warp * 16 + g + 8 * hh;
        if (!is_softmax || row >= Nl) continue;
        const float l = l_run[rb][hh];
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat16* op = a.out + b * a.o_b + (int64_t)(row0 + row) * a.o_n + h * a.o_h;
#pragma unroll
        for (int i = 0; i < 16; ++i)
          *reinterpret_cast<uint32_t*>(op + i * 8 + t4 * 2) =
              pack_bf16(o[rb][i][2 * hh] * inv, o[rb][i][2 * hh + 1] * inv);
        if (a.lse && t4 == 0)
          a.lse[((int64_t)b * a.H + h) * N + row0 + row] = (m_run[rb][hh] + log2f(l)) * kLn2;
      }
    }
    return;
  }

  // Merge across the cluster by pushing.  Rows [r*R, r*R + R) belong to block r.  A partial
  // row is 132 floats: 128 of O, then (max, sum).  Each block stages its rows in its own
  // shared memory and, once every block of the cluster is done with its operand tiles, sends
  // each owner its rows with ONE bulk shared-to-shared copy that signals the owner's mbarrier
  // (armed at start-up with the byte count it will receive).  Nobody waits on a remote round
  // trip; the owner reduces its C slots locally as soon as its mbarrier completes.
  const int C = a.C;
  const int rank = split % C;
  const int R = (Nl + C - 1) / C;
  float* sStage = reinterpret_cast<float*>(smem);                    // [Nl][kOStride]
  float* sRecv = sStage + (size_t)Nl * kOStride;                     // [C][R][kOStride]
#pragma unroll
  for (int rb = 0; rb < NB; ++rb) {
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int row = rb * 64 + warp * 16 + g + 8 * hh;
      if (!is_softmax || row >= Nl) continue;
      float* ro = sStage + row * kOStride;
#pragma unroll
      for (int i = 0; i < 16; ++i)
        *reinterpret_cast<float2*>(ro + i * 8 + t4 * 2) = make_float2(o[rb][i][2 * hh], o[rb][i][2 * hh + 1]);
      if (t4 == 0) *reinterpret_cast<float2*>(ro + kD) = make_float2(m_run[rb][hh], l_run[rb][hh]);
    }
  }
  fence_async_smem();                          // staged rows -> visible to the bulk-copy engine
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // every block's tiles are dead
  if (tid < C) {
    const int owner = tid;
    const int rows = max(0, min(R, Nl - owner * R));
    if (rows > 0) {
      const uint32_t src = smem_u32(sStage + (size_t)owner * R * kOStride);
      const uint32_t dst_local = smem_u32(sRecv + (size_t)rank * R * kOStride);
      uint32_t dst, rbar;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(dst_local), "r"(owner));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(bar_m), "r"(owner));
      asm volatile(
          "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
          ::"r"(dst), "r"(src), "r"((uint32_t)(rows * kOStride * 4)), "r"(rbar)
          : "memory");
    }
  }
  int merge_timeout = mbar_wait(bar_m, 0u) ? 0 : 1;
  // "I have received everything sent to me": once every block of the cluster has said so, all
  // copies out of this block's staged rows are complete too and it may leave (waited for at
  // the very end, after the reduction, when it has normally long completed)
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  const int sup = split / C;
  const int my_rows = max(0, min(R, Nl - rank * R));
  for (int idx = tid; idx < my_rows * 32; idx += kWsThreads) {
    const int lr = idx >> 5, mr = row0 + rank * R + lr, c4 = idx & 31;   // mr: global draft row
    float2 ml[kMaxCluster];
    float4 ov[kMaxCluster];
#pragma unroll
    for (int p = 0; p < kMaxCluster; ++p) {
      if (p < C) {
        const float* rr = sRecv + (size_t)(p * R + lr) * kOStride;
        ml[p] = *reinterpret_cast<const float2*>(rr + kD);
        ov[p] = *reinterpret_cast<const float4*>(rr + c4 * 4);
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int p = 0; p < kMaxCluster; ++p)
      if (p < C) M = fmaxf(M, ml[p].x);
    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float lsum = 0.f;
#pragma unroll
    for (int p = 0; p < kMaxCluster; ++p) {
      if (p < C) {
        const float w = (ml[p].x == -INFINITY) ? 0.f : ex2(ml[p].x - M);
        lsum += ml[p].y * w;
        o4.x += ov[p].x * w; o4.y += ov[p].y * w; o4.z += ov[p].z * w; o4.w += ov[p].w * w;
      }
    }
    if (a.Sp == 1) {
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      uint2 pk2;
      pk2.x = pack_bf16(o4.x * inv, o4.y * inv);
      pk2.y = pack_bf16(o4.z * inv, o4.w * inv);
      *reinterpret_cast<uint2*>(a.out + b * a.o_b + (int64_t)mr * a.o_n + h * a.o_h + c4 * 4) = pk2;
      if (a.lse && c4 == 0) a.lse[((int64_t)b * a.H + h) * N + mr] = (M + log2f(lsum)) * kLn2;
    } else {
      const int64_t base = ((((int64_t)b * a.H + h) * a.Sp + sup) * N + mr);
      *reinterpret_cast<float4*>(a.ws_o + base * kD + c4 * 4) = o4;
      if (c4 == 0) { a.ws_ml[base * 2] = M; a.ws_ml[base * 2 + 1] = lsum; }
    }
  }
  if (merge_timeout && tid == 0) atomicOr(&g_attn_error, 1u);
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// =======================================================================================
// Wide variant for N > 64 draft rows: one thread block covers 128 rows (N <= 256: one or two
// row blocks per head, adjacent in the grid so that they stream the same K/V tiles together).
//
// The tensor core needs the same time for an M = 64 and an M = 128 instruction, so two 64-row
// blocks per head spend twice the tensor time per K/V byte and the tensor pipe, not HBM,
// bounds N = 128.  Here S = Q K^T and O = P V are M = 128 instructions: accumulator row i lives
// in TMEM lane i, softmax warp w owns lanes 32w .. 32w+31 and every thread owns one whole row
// (no shuffles).  O stays in TMEM and accumulates across tiles; the running maximum used for the
// exponentials is only raised when a tile's maximum exceeds it by more than 2^8, and only then
// is the O row rescaled in TMEM (rare after the first tiles), so the per-tile work is
// load S, mask, exp2, pack P.  Probabilities are at most 2^8, harmless in bf16 / fp32.
// Key splits are merged inside a cluster of up to 8 blocks through distributed shared memory;
// only beyond 8 splits do the cluster results go to the caller's workspace for the combine kernel.
// =======================================================================================
constexpr int kWideQBytes = 128 * kRowBytes;            // 32 KB: 128 rows x 128 dims
constexpr int kWidePBytes = 128 * 128;                  // 16 KB: 128 rows x 64 keys
constexpr int kWideBarOffset = kWideQBytes + 2 * kTcStages * kTileBytes + kWidePBytes;   // 112 KB
__host__ __device__ constexpr int wide_smem_bytes() { return kWideBarOffset + kWsBarBytes; }
constexpr float kRescaleStep = 8.f;                     // log2 units

// 32 TMEM lanes (one per thread) x 32 consecutive columns
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// three-input maximum, and packed two-float multiply-add / add (one issue slot for two lanes)
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void fma2(float& x0, float& x1, float a0, float a1, float b, float c) {
  asm("{ .reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\t"
      "mov.b64 rb, {%4, %4};\n\t"
      "mov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
      "mov.b64 {%0, %1}, rd; }"
      : "=f"(x0), "=f"(x1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add2(float& acc0, float& acc1, float a0, float a1) {
  asm("{ .reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%0, %1};\n\t"
      "mov.b64 rb, {%2, %3};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\t"
      "mov.b64 {%0, %1}, rd; }"
      : "+f"(acc0), "+f"(acc1) : "f"(a0), "f"(a1));
}

// bits [shift, shift + 64) of a 256-bit row mask, zero outside [0, 256)
__device__ __forceinline__ unsigned long long mask_window(const unsigned long long (&m)[4], int shift) {
  if (shift <= -64 || shift >= 256) return 0ull;
  if (shift < 0) return m[0] << (-shift);
  const int wi = shift >> 6, r = shift & 63;
  const unsigned long long lo = wi == 0 ? m[0] : wi == 1 ? m[1] : wi == 2 ? m[2] : m[3];
  const unsigned long long hi = wi == 0 ? m[1] : wi == 1 ? m[2] : wi == 2 ? m[3] : 0ull;
  return r ? (lo >> r) | (hi << (64 - r)) : lo;
}

__global__ void __launch_bounds__(kWsThreads, 2)
tree_attention_wide_kernel(AttnArgs a, const __grid_constant__ CUtensorMap tm_q,
                           const __grid_constant__ CUtensorMap tm_k,
                           const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int N = a.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase;
  const uint32_t sK = sQ + kWideQBytes;
  const uint32_t sV = sK + kTcStages * kTileBytes;
  const uint32_t sP = sV + kTcStages * kTileBytes;
  const uint32_t bars = sbase + kWideBarOffset;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kWideBarOffset + kBarTmemSlot);
  volatile uint32_t* abort_word = reinterpret_cast<volatile uint32_t*>(smem + kWideBarOffset + kBarAbort);

  int bid = blockIdx.x;
  const int split = bid % a.S; bid = bid / a.S + a.unit0;
  const int rblk = bid % a.NBLK; bid /= a.NBLK;     // which 128-row block of the N draft rows
  // pack = 2 (N = 64, grouped KV heads): the block's 128 rows are the 64 draft rows of two query
  // heads that share one KV head, so that K/V stream is read once for both
  const int heads_per_block = a.pack;
  const int h0 = (bid % (a.H / heads_per_block)) * heads_per_block;
  const int b = bid / (a.H / heads_per_block);
  const int hk = h0 / a.group;
  const int row0 = rblk * 128;                       // first draft row of this thread block

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if ((sbase & 1023u) != 0) {   // the swizzled operand layout needs a 1024-byte aligned base
    if (tid == 0) atomicOr(&g_attn_error, 2u);
    return;                     // uniform over the grid: every block sees the same offset
  }

  if (tid == 0) {
    mbar_init(bars + kBarKFull, 1); mbar_init(bars + kBarKFull + 8, 1);
    mbar_init(bars + kBarVFull, 1); mbar_init(bars + kBarVFull + 8, 1);
    mbar_init(bars + kBarSFull, 1); mbar_init(bars + kBarSFull + 8, 1);
    mbar_init(bars + kBarOFull, 1);
    mbar_init(bars + kBarKFree, 1); mbar_init(bars + kBarKFree + 8, 1);
    mbar_init(bars + kBarVFree, 1); mbar_init(bars + kBarVFree + 8, 1);
    mbar_init(bars + kBarPFull, 4);            // one arrival per softmax warp
    mbar_init(bars + kBarQFull, 1);
    *abort_word = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // everything above is independent of the inputs; from here on global memory is read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int L = a.kv_len[b];
  const int total = L + N;
  const int ntiles = (total + kBN - 1) / kBN;
  const int t0 = tc_tile_begin(split, ntiles, a.S);
  const int t1 = tc_tile_begin(split + 1, ntiles, a.S);
  const int nt = t1 - t0;

  // softmax thread = draft row row0 + 32 warp + lane
  const int row = (warp & 3) * 32 + lane;            // row inside this block
  const int grow = heads_per_block == 2 ? (row & 63) : row0 + row;   // draft row
  const int h = heads_per_block == 2 ? h0 + (row >> 6) : h0;         // its query head
  float m_used = -INFINITY, l_run = 0.f;
  bool have_o = false;                 // this warp may read a finished O out of TMEM

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_warp = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      mbar_expect_tx(bars + kBarQFull, (uint32_t)kWideQBytes);
      // two 64-dim halves, each [128 rows x 128 B]; rows past N are zero-filled
      // second 64 rows: the next 64 draft rows of the same head, or the second head's rows
      const int r1 = heads_per_block == 2 ? 0 : row0 + 64, h1 = heads_per_block == 2 ? h0 + 1 : h0;
      tma_load_box(sQ, &tm_q, 0, row0, h0, b, a.q_slot, bars + kBarQFull);
      tma_load_box(sQ + 64 * 128, &tm_q, 0, r1, h1, b, a.q_slot, bars + kBarQFull);
      tma_load_box(sQ + 128 * 128, &tm_q, 64, row0, h0, b, a.q_slot, bars + kBarQFull);
      tma_load_box(sQ + 192 * 128, &tm_q, 64, r1, h1, b, a.q_slot, bars + kBarQFull);
    }
    // K tiles by lane 0, V tiles by lane 1: a K slot frees as soon as its Q K^T has run, a V slot
    // only after the softmax and P V of its tile; one thread issuing both in turn would hold the
    // next K tile back behind the wait for a V slot.
    if (lane < 2) {
      const bool is_v = lane == 1;
      const uint32_t ring = is_v ? sV : sK;
      const CUtensorMap* map = is_v ? &tm_v : &tm_k;
      const uint32_t full = bars + (is_v ? kBarVFull : kBarKFull), free_ = bars + (is_v ? kBarVFree : kBarKFree);
      int issued = 0;
      for (int it = 0; it < nt; ++it) {
        const int slot = it & 1, key0 = (t0 + it) * kBN;
        const uint32_t free_parity = (uint32_t)(((it >> 1) + 1) & 1);
        if (it >= 2 && !mbar_wait_abortable(free_ + slot * 8, free_parity, abort_word)) break;
        mbar_expect_tx(full + slot * 8, (uint32_t)kTileBytes);
        tma_load_box(ring + slot * kTileBytes, map, 0, key0, hk, b, a.kv_slot, full + slot * 8);
        tma_load_box(ring + slot * kTileBytes + 64 * 128, map, 64, key0, hk, b, a.kv_slot, full + slot * 8);
        ++issued;
      }
      if (*abort_word != 0u) {
        // giving up: let the copies already in flight land before this block goes away
        if (!is_v) mbar_wait(bars + kBarQFull, 0u);
        for (int it = max(0, issued - 2); it < issued; ++it)
          mbar_wait(full + (it & 1) * 8, (uint32_t)((it >> 1) & 1));
      }
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc(128, kBN, 0);
      constexpr uint32_t idesc_o = umma_idesc(128, kD, 1);
      const uint64_t dq0 = umma_desc(sQ, 16, 1024);
      const uint64_t dk0 = umma_desc(sK, 16, 1024);
      const uint64_t dp0 = umma_desc(sP, 16, 1024);
      const uint64_t dv0 = umma_desc(sV, kBN * 128, 1024);
      bool ok = mbar_wait_abortable(bars + kBarQFull, 0u, abort_word);
      // S[it & 1] = Q K(it)^T; that buffer's previous reader signalled P(it - 2) after reading it
      auto issue_qk = [&](int it) -> bool {
        const int slot = it & 1;
        if (!mbar_wait_abortable(bars + kBarKFull + slot * 8, (uint32_t)((it >> 1) & 1), abort_word)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t qoff = (uint32_t)((ks >> 2) * (128 * 128) + (ks & 3) * 32);
          const uint32_t koff = (uint32_t)((ks >> 2) * (64 * 128) + (ks & 3) * 32);
          umma_f16(tmem_base + kColS + slot * 64, dq0 + (qoff >> 4),
                   dk0 + ((slot * kTileBytes + koff) >> 4), idesc_s, ks > 0);
        }
        umma_commit(bars + kBarSFull + slot * 8);
        umma_commit(bars + kBarKFree + slot * 8);
        return true;
      };
      if (ok && nt > 0) ok = issue_qk(0);
      if (ok && nt > 1) ok = issue_qk(1);
      for (int it = 0; ok && it < nt; ++it) {
        const int slot = it & 1;
        // P(it) is in shared memory, and O has been rescaled if this tile raised the maximum
        if (!mbar_wait_abortable(bars + kBarPFull, (uint32_t)(it & 1), abort_word)) break;
        if (!mbar_wait_abortable(bars + kBarVFull + slot * 8, (uint32_t)((it >> 1) & 1), abort_word)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_f16(tmem_base + kColO, dp0 + ((kk * 32) >> 4),
                   dv0 + ((slot * kTileBytes + kk * 2048) >> 4), idesc_o, (it > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bars + kBarOFull);
        umma_commit(bars + kBarVFree + slot * 8);
        if (it + 2 < nt) ok = issue_qk(it + 2);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax warps
    // a wait's outcome is made warp-uniform, so the warp-wide TMEM instructions stay converged
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xFFFFFFFFu, mbar_wait_abortable(bar, parity, abort_word) ? 1 : 0) != 0;
    };
    bool ok = true;
    for (int it = 0; it < nt; ++it) {
      const int key0 = (t0 + it) * kBN;
      if (!wait_all(bars + kBarSFull + (it & 1) * 8, (uint32_t)((it >> 1) & 1))) { ok = false; break; }
      tc_fence_after();
      uint32_t s0[32], s1[32];
      tmem_ld_32x32(tmem_warp + kColS + (it & 1) * 64, s0);
      tmem_ld_32x32(tmem_warp + kColS + (it & 1) * 64 + 32, s1);
      tmem_wait_ld();
      // maximum of the raw scores (the scale is positive, so it commutes with max); the scale
      // is applied inside the exponent's multiply-add below
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // independent chains
      if (key0 + kBN <= L) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          mx4[j & 3] = max3(mx4[j & 3], __uint_as_float(s0[j]), __uint_as_float(s1[j]));
      } else {
        // "key j of this tile is visible to this row": prefix keys, then the row's tree bits
        // moved to where key L sits in this tile
        const int off = L - key0;                // position of key L in this tile (may be < 0)
        const unsigned long long pre = off >= 64 ? ~0ull : (off <= 0 ? 0ull : ((1ull << off) - 1ull));
        // the row's tree mask (up to 256 bits) is only needed here, in the last few tiles of a
        // context: read it from global memory (cached) rather than hold it in registers
        unsigned long long mrow[4] = {0ull, 0ull, 0ull, 0ull};
        if (grow < N) {
          const uint32_t* mp = a.mask + ((int64_t)b * N + grow) * a.Wm;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t w0 = 2 * i < a.Wm ? __ldg(mp + 2 * i) : 0u;
            const uint32_t w1 = 2 * i + 1 < a.Wm ? __ldg(mp + 2 * i + 1) : 0u;
            mrow[i] = (unsigned long long)w0 | ((unsigned long long)w1 << 32);
          }
        }
        const unsigned long long vis = pre | mask_window(mrow, -off);
        const uint32_t vlo = (uint32_t)vis, vhi = (uint32_t)(vis >> 32);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if (!((vlo >> j) & 1u)) s0[j] = 0xFF800000u;   // -inf
          if (!((vhi >> j) & 1u)) s1[j] = 0xFF800000u;
          mx4[j & 3] = max3(mx4[j & 3], __uint_as_float(s0[j]), __uint_as_float(s1[j]));
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
      // raise the reference maximum only when this tile exceeds it by more than the step
      bool o_done = it == 0;                      // "P V(it - 1) has completed" is known
      if (__any_sync(0xFFFFFFFFu, mx > m_used + kRescaleStep)) {
        const float m_new = fmaxf(m_used, mx);
        const float alpha = (m_new == -INFINITY) ? 1.f : ex2(m_used - m_new);   // m_used = -inf gives 0
        if (it > 0) {
          if (!wait_all(bars + kBarOFull, (uint32_t)((it - 1) & 1))) { ok = false; break; }
          tc_fence_after();
          o_done = true;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t orr[32];
            tmem_ld_32x32(tmem_warp + kColO + c * 32, orr);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) orr[j] = __float_as_uint(__uint_as_float(orr[j]) * alpha);
            tmem_st_32x32(tmem_warp + kColO + c * 32, orr);
          }
          tmem_wait_st();
        }
        l_run *= alpha;
        m_used = m_new;
      }
      const float ms = (m_used == -INFINITY) ? 0.f : m_used;
      uint32_t pk[32];
      float ps[4] = {0.f, 0.f, 0.f, 0.f};
      const float neg_ms = -ms;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        float x0, x1, x2, x3;
        fma2(x0, x1, __uint_as_float(s0[2 * j]), __uint_as_float(s0[2 * j + 1]), a.scale_log2, neg_ms);
        fma2(x2, x3, __uint_as_float(s1[2 * j]), __uint_as_float(s1[2 * j + 1]), a.scale_log2, neg_ms);
        pk[j] = pack_bf16(ex2(x0), ex2(x1));
        pk[16 + j] = pack_bf16(ex2(x2), ex2(x3));
        // the sum takes the rounded probabilities, the ones P V uses: with a lazily raised
        // maximum the largest probability is not exactly 1, and rounding it in the numerator
        // only would show up in peaked rows
        add2(ps[0], ps[1], __uint_as_float(pk[j] << 16), __uint_as_float(pk[j] & 0xFFFF0000u));
        add2(ps[2], ps[3], __uint_as_float(pk[16 + j] << 16), __uint_as_float(pk[16 + j] & 0xFFFF0000u));
      }
      l_run += (ps[0] + ps[1]) + (ps[2] + ps[3]);
      // the single P buffer is free once P V(it - 1) has completed
      if (!o_done && !wait_all(bars + kBarOFull, (uint32_t)((it - 1) & 1))) { ok = false; break; }
      if (key0 + kBN > total) {
        // Ragged last tile: rows of V past the last real key hold whatever the cache holds
        // there.  Their probabilities are zero, but 0 x NaN is NaN: clear them.
        if (!wait_all(bars + kBarVFull + (it & 1) * 8, (uint32_t)((it >> 1) & 1))) { ok = false; break; }
        const int first = total - key0;            // 0 < first < 64
        for (int c = tid; c < (kBN - first) * 16; c += 128) {
          const int vr = first + (c >> 4), chunk = c & 15;
          const uint32_t dst = sV + (it & 1) * kTileBytes + (chunk >> 3) * (64 * 128) + (vr >> 3) * 1024 +
                               (vr & 7) * 128 + (((chunk & 7) ^ (vr & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
        }
      }
      {
        // P row (64 bf16 = 8 chunks of 16 B) -> shared memory, K-major 128-byte-swizzled
        const uint32_t prow = sP + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(prow + ((c ^ (row & 7)) << 4)), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                         "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3])
                       : "memory");
      }
      fence_async_smem();                          // P (and cleared V rows) -> visible to the tensor core
      tc_fence_before();                           // this warp's TMEM accesses are done
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + kBarPFull);
    }
    have_o = ok && nt > 0 && wait_all(bars + kBarOFull, (uint32_t)((nt - 1) & 1));
    if (have_o) tc_fence_after();
  }

  const bool softmax_warp = warp < 4;
  const bool live = grow < N;
  if (a.C == 1) {
    // ---- no cluster: straight to the output, or (several clusters of one block never happen)
    if (softmax_warp && have_o) {
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t orr[32];
        __syncwarp();
        tmem_ld_32x32(tmem_warp + kColO + c * 32, orr);
        tmem_wait_ld();
        if (live) {
          __nv_bfloat16* op = a.out + b * a.o_b + (int64_t)grow * a.o_n + h * a.o_h + c * 32;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 pv;
            pv.x = pack_bf16(__uint_as_float(orr[8 * q4]) * inv, __uint_as_float(orr[8 * q4 + 1]) * inv);
            pv.y = pack_bf16(__uint_as_float(orr[8 * q4 + 2]) * inv, __uint_as_float(orr[8 * q4 + 3]) * inv);
            pv.z = pack_bf16(__uint_as_float(orr[8 * q4 + 4]) * inv, __uint_as_float(orr[8 * q4 + 5]) * inv);
            pv.w = pack_bf16(__uint_as_float(orr[8 * q4 + 6]) * inv, __uint_as_float(orr[8 * q4 + 7]) * inv);
            *reinterpret_cast<uint4*>(op + q4 * 8) = pv;
          }
        }
      }
      if (live && a.lse) a.lse[((int64_t)b * a.H + h) * N + grow] = (m_used + log2f(l_run)) * kLn2;
    }
  } else {
    // ---- merge across the cluster.  Rows [r*R, r*R + R) of this 128-row block belong to block
    // r.  After a first cluster barrier (every block's operand tiles are dead) each softmax
    // thread stores its row - 128 floats of O out of TMEM, then max and sum - straight into the
    // owner's shared memory (posted remote stores, slot = sender's rank); after a second barrier
    // each owner reduces its C slots locally.  Both barriers are passed by every thread of every
    // block whatever happened before, so a block that gave up cannot leave its mates waiting.
    const int C = a.C;
    const int rank = split % C;
    const int Nl = min(128, N - row0);
    const int R = (Nl + C - 1) / C;
    float* sRecv = reinterpret_cast<float*>(smem);                     // [C][R][kOStride]
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (softmax_warp) {
      const int owner = live ? row / R : 0;
      const uint32_t dst_local = smem_u32(sRecv + ((size_t)rank * R + (row - owner * R)) * kOStride);
      uint32_t dst;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(dst_local), "r"(owner));
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t orr[32];
        __syncwarp();
        if (have_o) {                       // warp-uniform
          tmem_ld_32x32(tmem_warp + kColO + c * 32, orr);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) orr[j] = 0u;
        }
        if (live) {
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};"
                         ::"r"(dst + (uint32_t)((c * 32 + q4 * 4) * 4)), "r"(orr[4 * q4]), "r"(orr[4 * q4 + 1]),
                           "r"(orr[4 * q4 + 2]), "r"(orr[4 * q4 + 3])
                         : "memory");
        }
      }
      if (live) {
        const float mm = have_o ? m_used : -INFINITY, ll = have_o ? l_run : 0.f;
        asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(dst + (uint32_t)(kD * 4)), "f"(mm), "f"(ll)
                     : "memory");
      }
    }
    tc_fence_before();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    const int sup = split / C;
    const int my_rows = max(0, min(R, Nl - rank * R));
    for (int idx = tid; idx < my_rows * 32; idx += kWsThreads) {
      const int lr = idx >> 5, mr = row0 + rank * R + lr, c4 = idx & 31;   // mr: draft row
      float2 ml[kMaxCluster];
      float4 ov[kMaxCluster];
#pragma unroll
      for (int p = 0; p < kMaxCluster; ++p) {
        if (p < C) {
          const float* rr = sRecv + (size_t)(p * R + lr) * kOStride;
          ml[p] = *reinterpret_cast<const float2*>(rr + kD);
          ov[p] = *reinterpret_cast<const float4*>(rr + c4 * 4);
        }
      }
      float M = -INFINITY;
#pragma unroll
      for (int p = 0; p < kMaxCluster; ++p)
        if (p < C) M = fmaxf(M, ml[p].x);
      float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
      float lsum = 0.f;
#pragma unroll
      for (int p = 0; p < kMaxCluster; ++p) {
        if (p < C) {
          const float w = (ml[p].x == -INFINITY) ? 0.f : ex2(ml[p].x - M);
          lsum += ml[p].y * w;
          o4.x += ov[p].x * w; o4.y += ov[p].y * w; o4.z += ov[p].z * w; o4.w += ov[p].w * w;
        }
      }
      if (a.Sp == 1) {
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        uint2 pk2;
        pk2.x = pack_bf16(o4.x * inv, o4.y * inv);
        pk2.y = pack_bf16(o4.z * inv, o4.w * inv);
        *reinterpret_cast<uint2*>(a.out + b * a.o_b + (int64_t)mr * a.o_n + h0 * a.o_h + c4 * 4) = pk2;
        if (a.lse && c4 == 0) a.lse[((int64_t)b * a.H + h0) * N + mr] = (M + log2f(lsum)) * kLn2;
      } else {
        const int64_t base = ((((int64_t)b * a.H + h0) * a.Sp + sup) * N + mr);
        *reinterpret_cast<float4*>(a.ws_o + base * kD + c4 * 4) = o4;
        if (c4 == 0) { a.ws_ml[base * 2] = M; a.ws_ml[base * 2 + 1] = lsum; }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_word != 0u && tid == 0) atomicOr(&g_attn_error, 1u);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }
}

// Merges the per-split partials: one warp per (context, head, row), 4 output dims per lane.
__global__ void __launch_bounds__(128)
tree_attention_combine_kernel(AttnArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t unit = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t nunits = (int64_t)a.B * a.H * a.N;
  if (unit >= nunits) return;
  const int row = (int)(unit % a.N);
  const int64_t bh = unit / a.N;
  const int h = (int)(bh % a.H);
  const int64_t b = bh / a.H;
  const float* pm = a.ws_ml + (bh * a.Sp * a.N + row) * 2;
  float M = -INFINITY;
  for (int s = 0; s < a.Sp; ++s) M = fmaxf(M, pm[(int64_t)s * a.N * 2]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float lsum = 0.f;
  for (int s = 0; s < a.Sp; ++s) {
    float ms = pm[(int64_t)s * a.N * 2], ls = pm[(int64_t)s * a.N * 2 + 1];
    float w = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
    lsum += ls * w;
    if (w != 0.f) {
      const float4 v = *reinterpret_cast<const float4*>(
          a.ws_o + ((bh * a.Sp + s) * a.N + row) * kD + lane * 4);
      acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
    }
  }
  const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
  __nv_bfloat16* op = a.out + b * a.o_b + row * a.o_n + h * a.o_h + lane * 4;
  uint2 pk;
  pk.x = pack_bf16(acc.x * inv, acc.y * inv);
  pk.y = pack_bf16(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(op) = pk;
  if (a.lse && lane == 0) a.lse[bh * a.N + row] = (M + log2f(lsum)) * kLn2;
}

// cuTensorMapEncodeTiled is reached through the runtime's driver entry point (no link against
// libcuda).  The maps describe bf16 tensors (d = 128, rows, heads, batch) with arbitrary 16-byte
// aligned strides; a box is 64 elements x 64 rows with 128-byte swizzle; out-of-range rows read
// as zeros.
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult st;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &st) != cudaSuccess ||
        st != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}
// A tensor map depends only on (base, extents, strides); a decoding loop passes the same few
// tensors call after call, so each host thread remembers the maps it has encoded in a small
// direct-mapped table and a repeated call costs a key comparison instead of a driver call.
struct MapKey {
  const void* base;
  int64_t rows, heads, batch, row_stride, head_stride, batch_stride;
  bool operator==(const MapKey& o) const {
    return base == o.base && rows == o.rows && heads == o.heads && batch == o.batch &&
           row_stride == o.row_stride && head_stride == o.head_stride && batch_stride == o.batch_stride;
  }
};
struct MapEntry { MapKey key; CUtensorMap map; int slot[3]; bool valid; };
constexpr int kMapCacheEntries = 256;

bool encode_box_map_uncached(CUtensorMap* map, const void* base, int64_t rows, int64_t heads, int64_t batch,
                             int64_t row_stride, int64_t head_stride, int64_t batch_stride, int (&slot)[3]);

bool encode_box_map(CUtensorMap* map, const void* base, int64_t rows, int64_t heads, int64_t batch,
                    int64_t row_stride, int64_t head_stride, int64_t batch_stride, int (&slot)[3]) {
  static thread_local MapEntry cache[kMapCacheEntries];
  const MapKey key{base, rows, heads, batch, row_stride, head_stride, batch_stride};
  uint64_t hsh = reinterpret_cast<uintptr_t>(base) >> 8;
  hsh = (hsh ^ (hsh >> 17) ^ (uint64_t)rows * 0x9E3779B97F4A7C15ull) * 0xD6E8FEB86659FD93ull;
  MapEntry& e = cache[(hsh >> 40) % kMapCacheEntries];
  if (e.valid && e.key == key) {
    *map = e.map;
    slot[0] = e.slot[0]; slot[1] = e.slot[1]; slot[2] = e.slot[2];
    return true;
  }
  if (!encode_box_map_uncached(map, base, rows, heads, batch, row_stride, head_stride, batch_stride, slot))
    return false;
  e.key = key; e.map = *map; e.valid = true;
  e.slot[0] = slot[0]; e.slot[1] = slot[1]; e.slot[2] = slot[2];
  return true;
}

bool encode_box_map_uncached(CUtensorMap* map, const void* base, int64_t rows, int64_t heads, int64_t batch,
                             int64_t row_stride, int64_t head_stride, int64_t batch_stride, int (&slot)[3]) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  // outer dimensions in order of increasing stride (size-1 dimensions last: their stride is unused)
  int64_t size[3] = {rows, heads, batch}, stride[3] = {row_stride, head_stride, batch_stride};
  int order[3] = {0, 1, 2};
  auto key = [&](int i) { return size[i] > 1 ? stride[i] : (int64_t)1 << 60; };
  for (int i = 0; i < 3; ++i)
    for (int j = i + 1; j < 3; ++j)
      if (key(order[j]) < key(order[i])) { int t = order[i]; order[i] = order[j]; order[j] = t; }
  cuuint64_t dims[4] = {(cuuint64_t)kD, 1, 1, 1};
  cuuint64_t strides[3] = {0, 0, 0};
  cuuint32_t box[4] = {64, 1, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  cuuint64_t prev = (cuuint64_t)kD * 2;
  for (int i = 0; i < 3; ++i) {
    const int which = order[i];
    slot[which] = i + 1;
    dims[i + 1] = (cuuint64_t)size[which];
    // the stride of a size-1 dimension never addresses anything: keep it legal and non-decreasing
    cuuint64_t st = size[which] > 1 ? (cuuint64_t)stride[which] * 2 : prev * dims[i];
    if (st < prev) st = prev;
    strides[i] = st;
    prev = st;
    if (which == 0) box[i + 1] = 64;
  }
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// How many clusters of c blocks of a kernel can be resident on the current device at once.
// The scheduler places a cluster inside one GPC, so this is not 2 * SMs / c: 37 clusters of 8
// do not fit although 296 blocks would, and the 37th cluster would run as a second wave.
// cudaOccupancyMaxActiveClusters knows the GPC layout but counts one block per SM for these
// kernels, while two are resident in practice; a cluster of c blocks at two per SM covers
// ceil(c / 2) SMs, so the number asked for is that of clusters of ceil(c / 2) blocks (all SMs
// for c <= 2).  Asked once per device, kernel and size; without a device (size queries on a
// machine that has none) the plain quotient stands in.
int cluster_capacity(bool wide, int c) {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cache[kMaxDev][2][kMaxCluster + 1];
  const int sms = rest::sm_count();
  const int nominal = (2 * (sms > 0 ? sms : 148)) / c;     // 148: size queries on a machine without a GPU
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { (void)cudaGetLastError(); return nominal; }
  const int have = cache[dev][wide ? 1 : 0][c].load(std::memory_order_relaxed);
  if (have > 0) return have;
  const int half = (c + 1) / 2;
  int n = 0;
  if (half == 1) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      return nominal;
    }
  } else {
    const void* fn = wide ? reinterpret_cast<const void*>(tree_attention_wide_kernel)
                          : reinterpret_cast<const void*>(tree_attention_ws_kernel);
    const size_t smem = wide ? (size_t)wide_smem_bytes() : (size_t)ws_smem_bytes();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(half * 64), 1, 1);
    cfg.blockDim = dim3((unsigned)kWsThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)half;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (rest::ensure_dynamic_smem(fn, wide ? rest::kSmemSlotAttnWide : rest::kSmemSlotAttn, smem) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      return nominal;
    }
  }
  cache[dev][wide ? 1 : 0][c].store(n, std::memory_order_relaxed);
  return n;
}

struct SplitPlan { int S, C, Sp; };

// Key splits per unit (context, head, row block).  The splits of a unit form clusters of C
// blocks (merged on chip); Sp clusters per unit (merged by the combine kernel when Sp > 1).
// The plan is the largest cluster size whose clusters all fit on the GPU at once - a partial
// second wave would double the time - then as many clusters per unit as still fit, and never
// more splits than tiles.
SplitPlan plan_splits(int B, int H, int N, int max_kv) {
  const int ntiles = (max_kv + kBN - 1) / kBN;
  const bool wide = N > 64;
  const int64_t units = (int64_t)B * H * (wide ? (N + 127) / 128 : 1);
  SplitPlan p;
  p.C = 1; p.S = 1; p.Sp = 1;
  for (int c = kMaxCluster; c >= 2; --c) {
    if (c > ntiles) continue;
    const int64_t cap = cluster_capacity(wide, c);
    if (units > cap) continue;
    int64_t sp = cap / units;
    if (sp > ntiles / c) sp = ntiles / c;
    if (sp > 64) sp = 64;
    if (sp < 1) sp = 1;
    p.C = c; p.Sp = (int)sp; p.S = c * (int)sp;
    break;
  }
  return p;
}

}  // namespace

extern "C" rest_status rest_device_error_flags(uint32_t* h_flags) {
  if (!h_flags) return REST_INVALID_ARG;
  unsigned int v = 0, zero = 0;
  REST_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_attn_error, sizeof(v)));
  if (v != 0) REST_CUDA_TRY(cudaMemcpyToSymbol(g_attn_error, &zero, sizeof(zero)));
  *h_flags = v;
  return REST_OK;
}

extern "C" rest_status rest_tree_attention_plan(int32_t B, int32_t H, int32_t N, int32_t D,
                                                int32_t max_kv, int32_t* out) {
  if (!out || B <= 0 || H <= 0 || N <= 0 || max_kv <= 0) return REST_INVALID_ARG;
  if (D != kD || N > REST_MAX_N) return REST_UNSUPPORTED;
  const SplitPlan p = plan_splits(B, H, N, max_kv);
  out[0] = p.S; out[1] = p.C; out[2] = p.Sp;
  out[3] = cluster_capacity(N > 64, p.C);
  return REST_OK;
}

extern "C" size_t rest_tree_attention_workspace_bytes(int32_t B, int32_t H, int32_t N, int32_t D,
                                                      int32_t max_kv) {
  if (B <= 0 || H <= 0 || N <= 0 || D != kD || max_kv <= 0) return 0;
  const SplitPlan p = plan_splits(B, H, N, max_kv);
  if (p.Sp == 1) return 0;
  return (size_t)B * H * p.Sp * N * (kD + 2) * sizeof(float);
}

extern "C" rest_status rest_tree_attention(const void* d_q, const void* d_k, const void* d_v,
                                           const int64_t* strides, const int32_t* d_kv_len,
                                           const uint32_t* d_mask, int32_t B, int32_t H,
                                           int32_t H_kv, int32_t N, int32_t D, int32_t max_kv,
                                           float scale, void* d_out, float* d_lse, void* d_ws,
                                           size_t ws_bytes, void* stream) {
  if (B < 0 || H < 1 || H_kv < 1 || N < 1 || max_kv < 1 || !strides) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_q || !d_k || !d_v || !d_kv_len || !d_mask || !d_out) return REST_INVALID_ARG;
  if (!(scale > 0.f) || !(scale < INFINITY)) return REST_INVALID_ARG;
  if (D != kD || N > REST_MAX_N || (H % H_kv) != 0) return REST_UNSUPPORTED;
  for (int i = 0; i < 9; ++i)
    if (strides[i] < 0 || (strides[i] % 8) != 0) return REST_INVALID_ARG;
  {
    // a dimension that is actually stepped through must advance by at least one row of D elements
    const int64_t extent[9] = {B, N, H, B, H_kv, max_kv, B, N, H};
    for (int i = 0; i < 9; ++i)
      if (extent[i] > 1 && strides[i] < D) return REST_INVALID_ARG;
  }
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k) |
       reinterpret_cast<uintptr_t>(d_v) | reinterpret_cast<uintptr_t>(d_out)) & 15)
    return REST_INVALID_ARG;
  if ((int64_t)B * H * 64 > 0x7FFFFFFFll) return REST_UNSUPPORTED;

  AttnArgs a;
  a.q = static_cast<const __nv_bfloat16*>(d_q);
  a.k = static_cast<const __nv_bfloat16*>(d_k);
  a.v = static_cast<const __nv_bfloat16*>(d_v);
  a.out = static_cast<__nv_bfloat16*>(d_out);
  a.lse = d_lse; a.kv_len = d_kv_len; a.mask = d_mask;
  a.q_b = strides[0]; a.q_n = strides[1]; a.q_h = strides[2];
  a.kv_b = strides[3]; a.kv_h = strides[4]; a.kv_l = strides[5];
  a.o_b = strides[6]; a.o_n = strides[7]; a.o_h = strides[8];
  a.B = B; a.H = H; a.group = H / H_kv; a.N = N; a.Wm = (N + 31) / 32;
  const SplitPlan plan = plan_splits(B, H, N, max_kv);
  a.S = plan.S; a.C = plan.C; a.Sp = plan.Sp;
  a.scale_log2 = scale * kLog2e;
  a.ws_o = nullptr; a.ws_ml = nullptr;
  if (a.Sp > 1) {
    size_t need = rest_tree_attention_workspace_bytes(B, H, N, D, max_kv);
    if (!d_ws) return REST_INVALID_ARG;
    if (ws_bytes < need) return REST_WORKSPACE_TOO_SMALL;
    a.ws_o = static_cast<float*>(d_ws);
    a.ws_ml = a.ws_o + (size_t)B * H * a.Sp * N * kD;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Grouped KV heads with N = 64 and a batch that fills the GPU without key splits: two query
  // heads of a group share one 128-row block of the wide kernel (their K/V is streamed once)
  a.pack = (N == 64 && (a.group % 2) == 0 && (int64_t)B * H / 2 >= 2 * rest::sm_count()) ? 2 : 1;
  const bool wide = N > 64 || a.pack == 2;
  a.NBLK = N > 64 ? (N + 127) / 128 : 1;
  const size_t smem = wide ? (size_t)wide_smem_bytes() : (size_t)ws_smem_bytes();
  if (wide)
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(tree_attention_wide_kernel), rest::kSmemSlotAttnWide, smem));
  else
    REST_CUDA_TRY(rest::ensure_dynamic_smem(reinterpret_cast<const void*>(tree_attention_ws_kernel), rest::kSmemSlotAttn, smem));
  if ((int64_t)B * H * a.NBLK * a.S > 0x7FFFFFFFll) return REST_UNSUPPORTED;
  // Units that need no key split but do not fill a whole number of waves: the units of the last,
  // partial wave go into a second launch with their key range cut over one cluster each, so that
  // the wave ends after a fraction of a full block's time instead of a whole one.  Worth it when
  // a block has enough tiles for the saving to exceed the merge and the launch.
  const int64_t units = (int64_t)B * (H / a.pack) * a.NBLK;
  const int64_t slots = 2 * (int64_t)cluster_capacity(wide, 1);
  const int ntiles_max = (max_kv + kBN - 1) / kBN;
  int64_t tail_units = 0;
  int tail_c = 1;
  if (a.S == 1 && a.pack == 1 && units > slots && ntiles_max >= 16) {
    const int64_t r = units % slots;
    if (r > 0) {
      for (int c = kMaxCluster; c >= 2; --c) {
        if (r <= cluster_capacity(wide, c)) { tail_units = r; tail_c = c; break; }
      }
    }
  }
  a.unit0 = 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((units - tail_units) * a.S), 1, 1);
  cfg.blockDim = dim3((unsigned)kWsThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)a.C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // the kernel waits (griddepcontrol.wait) before its first global access, so it may be
  // launched while the kernel before it in the stream is still draining
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // tensor maps: Q (d, N rows, H, B); K and V (d, max_kv rows, H_kv, B)
  CUtensorMap tm_q, tm_k, tm_v;
  int v_slot[3];
  if (!encode_box_map(&tm_q, d_q, N, H, B, a.q_n, a.q_h, a.q_b, a.q_slot) ||
      !encode_box_map(&tm_k, d_k, max_kv, H_kv, B, a.kv_l, a.kv_h, a.kv_b, a.kv_slot) ||
      !encode_box_map(&tm_v, d_v, max_kv, H_kv, B, a.kv_l, a.kv_h, a.kv_b, v_slot))
    return rest::note_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  if (wide)
    REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, tree_attention_wide_kernel, a, tm_q, tm_k, tm_v));
  else
    REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, tree_attention_ws_kernel, a, tm_q, tm_k, tm_v));
  rest::count_launch();
  if (tail_units > 0) {
    AttnArgs t = a;
    t.unit0 = (int)(units - tail_units);
    t.S = tail_c; t.C = tail_c; t.Sp = 1;
    cfg.gridDim = dim3((unsigned)(tail_units * tail_c), 1, 1);
    attr[0].val.clusterDim.x = (unsigned)tail_c;
    if (wide)
      REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, tree_attention_wide_kernel, t, tm_q, tm_k, tm_v));
    else
      REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, tree_attention_ws_kernel, t, tm_q, tm_k, tm_v));
    rest::count_launch();
  }
  if (a.Sp > 1) {
    const int64_t rows = (int64_t)B * H * N;
    tree_attention_combine_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(a);
    rest::count_launch();
    REST_CUDA_TRY(cudaGetLastError());
  }
  return REST_OK;
}

// ---------------------------------------------------------------------------------------
// Variant for callers that cannot allocate device memory.
//
// The split partials live in a fixed array that is part of the library image, so the caller
// passes no workspace.  The array is a device symbol: its name is only meaningful in device
// code, so host code asks the runtime for its device address once per device (with that
// device current) and hands that address to the unchanged rest_tree_attention.
// ---------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = REST_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_static_scratch_addr[kMaxDevices];   // device address of g_static_scratch, per device

rest_status static_scratch_pointer(void** out) {
  int dev = 0;
  REST_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return REST_UNSUPPORTED;
  void* p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    // two threads may both ask the first time; they get the same address
    REST_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    g_static_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return REST_OK;
}

}  // namespace

extern "C" rest_status rest_tree_attention_static_scratch(
    const void* d_q, const void* d_k, const void* d_v, const int64_t* strides,
    const int32_t* d_kv_len, const uint32_t* d_mask, int32_t B, int32_t H, int32_t H_kv, int32_t N,
    int32_t D, int32_t max_kv, float scale, void* d_out, float* d_lse, void* stream) {
  const size_t need = rest_tree_attention_workspace_bytes(B, H, N, D, max_kv);
  if (need > kStaticScratchBytes) return REST_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  rest_status st = static_scratch_pointer(&scratch);
  if (st != REST_OK) return st;
  return rest_tree_attention(d_q, d_k, d_v, strides, d_kv_len, d_mask, B, H, H_kv, N, D, max_kv,
                             scale, d_out, d_lse, scratch, kStaticScratchBytes, stream);
}
