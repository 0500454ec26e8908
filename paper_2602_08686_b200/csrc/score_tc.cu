// Tensor-core window-score scan for bf16 inputs on sm_100a (Sec. 3 softmax; Eq. 4 window mass).
//
// One persistent, warp-specialised kernel does both passes over K:
//   P1 (row statistics)  D[row, key]  = Q_blk . K_tile^T   (UMMA M = 128 query rows, N = 128 keys):
//        one TMEM lane per query row, so the running row maximum and the sum of exponentials are
//        thread-local; per-run partial pairs go to global memory and the last warp to finish a chunk
//        merges them in a fixed order into (max, max + log2 sum).
//   P2 (column sums)     D[key, row]  = K_tile . Q_blk^T   (the same shared-memory tiles, operands
//        swapped): one TMEM lane per key, so c_h[t] = sum_i 2^(x[i,t] - bias_i) is thread-local.
// A "chunk" is one (unit, KV head, block of 128 query rows); a "run" is a few consecutive key tiles of
// a chunk.  CTAs take runs from two global queues (atomic counters), one per pass, in run order: P1
// runs can always be taken; a P2 run can start once its chunk's statistics are final, which happens
// shortly after the chunk's last P1 run.  By then the other CTAs have streamed far more than L2 retains, so
// the second read of a K tile comes from HBM as well (L2 serves the query blocks and the partial statistics).
// Results do not depend on which CTA takes which run.  Warp roles:
//   warp 0       producer (one thread): hands runs to two "lanes" (the even and the odd sub-items),
//                issues the TMA loads and describes every sub-item (one tile of one pass) to the others
//                through a descriptor ring in shared memory.  Sub-item j uses K stage j % 5, TMEM buffer
//                j % 4 and the Q buffer of lane j % 2.  The odd lane prefers P2 runs and the even lane P1
//                runs; a lane whose preferred queue has nothing ready takes a run of the other pass.
//   warps 1, 19  MMA issuers (one thread each, even / odd j): tcgen05.mma M = N = K = 128 into one of four
//                128-column TMEM buffers.
//   warps 2..17  consumers: four groups, one per TMEM buffer, each with one warp per lane quadrant,
//                read the accumulators back with tcgen05.ld.
//   warp 18      scout: reserves the CTA's next P2 runs, waits for their chunks' statistics and stages
//                their 128 row biases in shared memory.
// K and Q tiles arrive by TMA (128-byte swizzle) and feed tcgen05.mma directly.
//
// Every wait is bounded: an mbarrier or flag wait that exceeds its time limit records a code in the
// work space's status word (reported as CKV_ERR_TIMEOUT) and the CTA winds down (frees TMEM, returns).
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <type_traits>
#include <string>

#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kTile = 128;        // keys per tile, also query rows per block
constexpr int kStages = 5;        // K-tile ring
constexpr int kFullBars = 2 * kStages;
constexpr int kTmemBufs = 4;      // accumulator buffers of 128 columns, one per consumer group
constexpr int kRing = 16;         // descriptor slots
static_assert(kRing >= kStages + kTmemBufs, "a descriptor slot is reused only after its readers are done");
constexpr int kBiasBufs = 4;      // bias vectors of the most recent P2 chunks
constexpr int kConsumerWarps = 16;
constexpr int kScoutWarp = 2 + kConsumerWarps;
constexpr int kMma2Warp = 3 + kConsumerWarps;
constexpr int kThreads = 32 * (4 + kConsumerWarps);
constexpr uint32_t kHalfBytes = 128 * 128;          // 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfBytes;     // 128 rows x 128 bf16
constexpr float kMinRowMax = -1.0e30f;              // stands in for "no visible key yet"

// x = (q.k) * log2(e) / sqrt(128)
constexpr float kScale = 0.12751743074602467f;

// UMMA instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);


struct TcArgs {
  int Nu, H, Hkv, G, L, W, n;
  int RB, hpb;          // row blocks per KV group; query heads per row block (128 / W)
  int T, run, RPC, C;   // key tiles per chunk; tiles per run; runs per chunk; chunks
  int NR;               // runs in total
  int ppr, expected;    // partial pairs per run (1 or 2); pairs per (chunk, lane quadrant)
  int hints;
  uint32_t q_bytes;     // bytes of one Q block load
  int q_split;          // the Q box holds fewer than 128 rows: its two halves are loaded separately
  float* csum;
  // Grouped output (a KV group's query heads fill one row block, max or no pooling): instead of the
  // per-head column sums c_h[t], P2 writes zgrp[u, g, t] = max_h head_w[h] * ((L / W) c_h[t]) and
  // mgrp[u, g, t] = sum_h c_h[t] (heads in index order); both are [Nu, Hkv, L].  Null zgrp: per-head output.
  float* zgrp;
  float* mgrp;
  const float* head_w;
  int64_t hw_stride;    // elements between the head tables of consecutive units (0: one shared table)
  float lw_scale;       // L / W
  float2* part;         // [C][ppr*RPC][128] partial (row max, row sum) per run and consumer group
  float2* stat;         // [C][128]          (row max, row max + log2 row sum)
  int* done;            // [C][4]
  int* ready;           // [C]
  int* queue;           // [2] next P1 run and next P2 run to hand out
  int* status;
  unsigned long long wait_ns;   // time limit of every wait
};

// What the producer tells the other warps about sub-item j (ring slot j % kRing).
enum : int { kP1 = 0, kP2 = 1, kNop = 2, kStop = 3 };
struct __align__(16) Desc {
  int type;       // kP1, kP2, kNop, kStop; bit 9: phase parity of the stream's q_full barrier to wait for
  int chunk;
  int tile;       // key tile within the chunk
  int part_slot;  // P1: where this group's pair of the run goes, or -1 while the run goes on
                  // P2: offset of the row block's first head in the head-weight table
  int first;      // P1: this group's first tile of the run (reset the running pair)
                  // P2: index (u * Hkv + g) of the KV group
  int head0;      // P2: index (u * H + head) of the first query head of the row block
  int n_heads;    // query heads of the row block that exist
  int nbias_buf;  // P2: which bias vector belongs to the tile's chunk
};

// ------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.b32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait on an mbarrier phase.  Returns false after the time limit (or when another warp of
// the CTA already gave up), having recorded the failure.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                            int code, unsigned long long limit_ns) {
  const unsigned long long t0 = global_ns();
  for (int it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255) == 255) {
      if (*abort_flag) {
        atomicCAS(status + 1 + (code & 7), 0, code);  // which wait each role was in when the CTA gave up
        return false;
      }
      if (global_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          int code, unsigned long long limit_ns) {
  for (int it = 0; it < 64; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, code, limit_ns);
}

__device__ __forceinline__ void tma_load_5d(const CUtensorMap* map, uint32_t dst, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4),
      "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand with 128-byte swizzle (rows 128 bytes apart,
// groups of eight rows 1024 bytes apart, descriptor version 1), split into its address field (low
// word: smem address / 16 in the low 14 bits, leading byte offset 1) and the constant rest, so that
// stepping through a tile is one integer add.
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t addr) { return ((addr >> 4) & 0x3fffu) | (1u << 16); }
__device__ __forceinline__ uint64_t umma_desc_from_lo(uint32_t lo) {
  constexpr uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two-wide fp32 arithmetic (one instruction for a pair of values) and a three-input maximum: the
// consumer loops are bound by instruction issue, and these halve the multiply-add, add and max counts.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// What one of the two slot lanes (even / odd sub-items) is working on: a run of either pass, and the
// state of the lane's Q buffer.
struct Lane {
  int type, k, tr, chunk, ric, u, g, head0, heads, gen;   // the run in hand (k == tr: none)
  int q_chunk, q_last, q_loads;  // chunk whose rows the lane's Q buffer holds; its last reader; loads so far
  __device__ void init() {
    type = kNop, k = 0, tr = 0, chunk = -1, ric = 0, u = 0, g = 0, head0 = 0, heads = 1, gen = 0;
    q_chunk = -1, q_last = -1000, q_loads = 0;
  }
  // Takes global run rho of pass ty and works out where its chunk lives.
  __device__ void take(const TcArgs& a, int rho, int ty, int generation) {
    type = ty, k = 0, gen = generation;
    const int c = rho / a.RPC;
    ric = rho - c * a.RPC;
    tr = min(a.run, a.T - ric * a.run);
    if (c != chunk) {
      chunk = c;
      const int per_unit = a.Hkv * a.RB;
      u = c / per_unit;
      const int g_rb = c - u * per_unit;
      g = g_rb / a.RB;
      const int rb = g_rb - g * a.RB;
      head0 = g * a.G + rb * a.hpb;
      heads = min(a.hpb, a.G - rb * a.hpb);
    }
  }
};

// ------------------------------------------------------------------------------------ shared memory
struct __align__(1024) Smem {
  uint8_t k[kStages][kTileBytes];  // K tiles: two 64-column halves of [128 rows][128 bytes], swizzled
  uint8_t q[2][kTileBytes];        // query rows of the run on the even lane and of the run on the odd lane
  float nbias[kBiasBufs][kTile];   // negated row biases -(max + log2 sum) of the most recent P2 runs
  Desc desc[kRing];
  // full[j % kFullBars] says sub-item j's K tile has landed.  There are two barriers per K stage so that
  // each of the two MMA threads (even / odd j) sees every phase of the barriers it waits on: a parity wait
  // is only sound for a waiter that never skips a phase.
  uint64_t full[kFullBars], empty[kStages], tmem_full[kTmemBufs], tmem_empty[kTmemBufs];
  uint64_t q_full[2];              // a lane's Q rows have landed
  uint32_t tmem_base;
  int abort_flag;
  int p2_ready_gen;   // scout -> producer: P2 runs ("generations", counted from 1) up to this one are staged ...
  int p2_rho[kBiasBufs];       // ... which global run each of them is, per generation % kBiasBufs ...
  int p2_total;       // ... and how many there will be in all (-1 until the scout knows)
  int gen_fin[kBiasBufs];      // producer -> scout: generation whose last tile was issued, per generation % kBiasBufs ...
  int gen_last_j[kBiasBufs];   // ... and the sub-item index of that last tile
  int prod_j;         // producer -> scout: index of the sub-item being issued
};
static_assert(sizeof(Smem) <= 232448, "shared memory of one CTA");

// One 32-column slice of an accumulator tile, with the causal / end-of-sequence mask of a P1 row
// applied when the tile reaches past the prefix: keys t > limit are hidden (-inf).
__device__ __forceinline__ void load_logits(uint32_t taddr, float (&v)[32], bool tail, int tbase, int limit) {
  tmem_ld32(taddr, v);
  if (tail) {
#pragma unroll
    for (int jj = 0; jj < 32; ++jj)
      if (tbase + jj > limit) v[jj] = -INFINITY;
  }
}

// Merge of `count` partial (max, sum) pairs of one row, 1 KB apart, in slot order.
__device__ __forceinline__ float2 merge_pairs(const float2* p, int count) {
  float m = kMinRowMax, l = 0.f;
  int sl = 0;
  for (; sl + 32 <= count; sl += 32) {  // all loads of a batch in flight together
    float2 pr[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) pr[e] = __ldcg(p + (int64_t)(sl + e) * kTile);
    float bm = pr[0].x;
#pragma unroll
    for (int e = 1; e < 32; ++e) bm = fmaxf(bm, pr[e].x);
    const float mn = fmaxf(m, bm);
    float acc = l * ex2(m - mn);
#pragma unroll
    for (int e = 0; e < 32; ++e) acc += pr[e].y * ex2(pr[e].x - mn);
    m = mn, l = acc;
  }
  for (; sl < count; ++sl) {
    const float2 pr = __ldcg(p + (int64_t)sl * kTile);
    const float mn = fmaxf(m, pr.x);
    l = l * ex2(m - mn) + pr.y * ex2(pr.x - mn);
    m = mn;
  }
  return make_float2(m, l);
}

// kGrouped: pass 2 writes the per-group maximum and mass (TcArgs::zgrp) instead of per-head column sums.
template <int W, bool kGrouped>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map, TcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  if (smem_u32(smem_raw) & 1023u) {  // the swizzled tiles need 1024-byte alignment; never seen, but checked
    if (threadIdx.x == 0) atomicCAS(a.status, 0, 41);
    return;
  }
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&sm.empty[s]), 1);
    for (int s = 0; s < kFullBars; ++s) mbar_init(smem_u32(&sm.full[s]), 1);
    for (int b = 0; b < kTmemBufs; ++b) {
      mbar_init(smem_u32(&sm.tmem_full[b]), 1);
      mbar_init(smem_u32(&sm.tmem_empty[b]), 4);
    }
    mbar_init(smem_u32(&sm.q_full[0]), 1);
    mbar_init(smem_u32(&sm.q_full[1]), 1);
    sm.abort_flag = 0;
    sm.p2_ready_gen = 0;
    sm.p2_total = -1;
    for (int e = 0; e < kBiasBufs; ++e) sm.gen_fin[e] = 0, sm.gen_last_j[e] = 0, sm.p2_rho[e] = 0;
    sm.prod_j = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sm.tmem_base;
  const int NR = a.NR;
  int* const queue = a.queue;

  if (warp == 0) {
    // ================================================================= producer: schedule + TMA (one thread)
    if (lane == 0) {
      Lane ln0, ln1;       // even and odd sub-items
      ln0.init(), ln1.init();
      int gen = 0;         // P2 runs started so far; the biases of run e live in nbias[e % kBiasBufs]
      int p1_next = atomicAdd(queue, 1);   // the CTA's next P1 run, fetched one run ahead
      const uint64_t pol_q = policy_evict_last();
      const uint64_t pol_k0 = a.hints ? policy_evict_last() : policy_evict_normal();
      const uint64_t pol_k1 = a.hints ? policy_evict_first() : policy_evict_normal();
      bool ok = true;
      int j = 0;
      unsigned long long t_busy = global_ns();   // when the producer last had a tile to issue
      auto p2_done = [&] { return gen == *(volatile int*)&sm.p2_total; };
      // Hands the lane its next run.  The even lane prefers P1 and the odd lane P2, so that in the steady
      // state the two passes alternate; a lane whose preferred queue has nothing to give (no P2 run whose
      // chunk is final, or no P1 run left) takes a run of the other pass instead of idling.
      auto refill = [&](Lane& ln, const bool prefer_p2) {
        const bool p2_ok = *(volatile int*)&sm.p2_ready_gen >= gen + 1;   // the scout has staged the next P2 run
        const bool p1_ok = p1_next < NR;
        if (p2_ok && (prefer_p2 || !p1_ok)) {
          __threadfence_block();
          ++gen;
          ln.take(a, *(volatile int*)&sm.p2_rho[gen % kBiasBufs], kP2, gen);
        } else if (p1_ok) {
          ln.take(a, p1_next, kP1, 0);
          p1_next = atomicAdd(queue, 1);
        }
      };
      // Issues the next tile of the lane's run as sub-item j.
      auto issue = [&](Lane& ln, const int lane_id) {
        const int stage = j % kStages;
        const uint32_t bar = smem_u32(&sm.full[j % kFullBars]);
        int4* d = reinterpret_cast<int4*>(&sm.desc[j % kRing]);
        const bool reload = ln.chunk != ln.q_chunk;
        if (reload) {
          // The MMAs that read the lane's old rows must have completed (they all come from the lane's own
          // MMA thread, in order).  The wait on this sub-item's K stage covers sub-items up to
          // j - kStages; a younger reader needs its own stage's barrier.
          if (ln.q_last > j - kStages)
            ok = mbar_wait(smem_u32(&sm.empty[ln.q_last % kStages]), (ln.q_last / kStages) & 1, abort_flag, a.status,
                           12 | (j << 8), a.wait_ns);
          if (!ok) return;
          ++ln.q_loads;
          ln.q_chunk = ln.chunk;
        }
        ln.q_last = j;
        const int tile = ln.ric * a.run + ln.k;
        // the n-th load of a lane's rows (n = 0, 1, ...) completes phase n of its barrier: wait for parity n & 1
        const int q_phase = (ln.q_loads - 1) & 1;
        if (ln.type == kP1) {
          d[0] = make_int4(ln.type | (q_phase << 9), ln.chunk, tile,
                           (ln.k + 2 >= ln.tr) ? ln.ric * a.ppr + (ln.k & 1) : -1);
          d[1] = make_int4(ln.k < 2, 0, ln.heads, 0);
        } else {
          d[0] = make_int4(ln.type | (q_phase << 9), ln.chunk, tile, ln.u * (int)a.hw_stride + ln.head0);
          d[1] = make_int4(ln.u * a.Hkv + ln.g, ln.u * a.H + ln.head0, ln.heads, ln.gen % kBiasBufs);
        }
        mbar_arrive_expect_tx(bar, kTileBytes);
        if (reload) {
          const uint32_t qbar = smem_u32(&sm.q_full[lane_id]);
          mbar_arrive_expect_tx(qbar, a.q_bytes);
          tma_load_5d(&q_map, smem_u32(sm.q[lane_id]), qbar, 0, 0, ln.head0, 0, ln.u, pol_q);
          if (a.q_split)
            tma_load_5d(&q_map, smem_u32(sm.q[lane_id]) + kHalfBytes, qbar, 0, 0, ln.head0, 1, ln.u, pol_q);
        }
        tma_load_5d(&k_map, smem_u32(sm.k[stage]), bar, 0, tile * kTile, 0, ln.g, ln.u,
                    ln.type == kP1 ? pol_k0 : pol_k1);
        if (++ln.k == ln.tr && ln.type == kP2) {
          // the run's biases may be replaced once its readers are done: tell the scout where it ended
          *(volatile int*)&sm.gen_last_j[ln.gen % kBiasBufs] = j;
          __threadfence_block();
          *(volatile int*)&sm.gen_fin[ln.gen % kBiasBufs] = ln.gen;
        }
      };
      while (ok) {
        if (ln0.k == ln0.tr && ln1.k == ln1.tr && p1_next >= NR && p2_done()) break;
        int idle = 0;
#pragma unroll
        for (int slot = 0; slot < 2; ++slot, ++j) {
          Lane& ln = slot == 0 ? ln0 : ln1;
          if (ln.k == ln.tr) refill(ln, slot == 1);
          ok = ok && mbar_wait(smem_u32(&sm.empty[j % kStages]), ((j / kStages) & 1) ^ 1, abort_flag, a.status,
                               11 | (j << 8), a.wait_ns);
          if (!ok) break;
          *(volatile int*)&sm.prod_j = j;
          if (ln.k < ln.tr) {
            issue(ln, slot);
          } else {
            ++idle;
            sm.desc[j % kRing].type = kNop;
            mbar_arrive(smem_u32(&sm.full[j % kFullBars]));
          }
          if (!ok) break;
        }
        if (idle == 2) {  // nothing to issue on either lane: P2 runs are waiting for their chunks
          __nanosleep(200);
          if (*abort_flag) {
            ok = false;
          } else if (global_ns() - t_busy > a.wait_ns) {
            *abort_flag = 1;
            atomicCAS(a.status, 0, 16 | (j << 8));
            ok = false;
          }
        } else {
          t_busy = global_ns();
        }
      }
      // one stop marker per consumer group
      for (int e = 0; e < kTmemBufs && ok; ++e, ++j) {
        ok = mbar_wait(smem_u32(&sm.empty[j % kStages]), ((j / kStages) & 1) ^ 1, abort_flag, a.status, 14 | (j << 8), a.wait_ns);
        if (ok) {
          sm.desc[j % kRing].type = kStop;
          mbar_arrive(smem_u32(&sm.full[j % kFullBars]));
        }
      }
      if (!ok) {
        // give copies in flight time to land before the CTA's shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == kScoutWarp) {
    // ================================================================= scout: stages the biases of the P2 runs
    // Reserves P2 runs from the global queue, a window of kBiasBufs at a time (lane i looks after the run
    // that will be this CTA's generation G + i), polls the readiness flags of their chunks together, and
    // stages them in order: copies the negated biases into shared memory and tells the producer which
    // run it is.
    unsigned long long t_progress = global_ns();
    bool ok = true;
    int G = 1;          // next generation to stage
    // run reserved for generation G + lane: the first window in one step, so that it is in increasing order
    // (later reservations are made one at a time and the counter only grows)
    int my_rho = 0;
    if (lane == 0) my_rho = atomicAdd(queue + 1, kBiasBufs);
    my_rho = __shfl_sync(0xffffffffu, my_rho, 0) + lane;   // every lane takes part in the shuffle
    if (lane >= kBiasBufs) my_rho = NR;
    bool mine = false;  // its chunk is known to be final
    int it = 0;
    while (ok) {
      const int rho0 = __shfl_sync(0xffffffffu, my_rho, 0);
      if (rho0 >= NR) break;   // the queue is exhausted (runs are handed out in increasing order)
      if (!mine && my_rho < NR) mine = ld_acquire(a.ready + my_rho / a.RPC) >= 4;
      const unsigned ready_mask = __ballot_sync(0xffffffffu, mine);
      bool staged = false;
      if (ready_mask & 1u) {
        // nbias[G % kBiasBufs] last served run G - kBiasBufs: all of its tiles must have been issued, and a
        // tile's readers are done once the producer has got kStages + 2 kTmemBufs sub-items past it (it waits
        // for the K stage of sub-item j - kStages to be free, whose MMA waited for the release of the TMEM
        // buffer by sub-item j - kStages - kTmemBufs; a warp releases a sub-item's buffer after its last
        // accumulator load and before that slice's math, so what is certain then is that it has finished
        // all math, bias reads included, of its sub-item before, j - kStages - 2 kTmemBufs).
        bool free_buf = true;
        if (G > kBiasBufs) {
          free_buf = *(volatile int*)&sm.gen_fin[G % kBiasBufs] == G - kBiasBufs;
          if (free_buf) {
            __threadfence_block();
            free_buf = *(volatile int*)&sm.prod_j >= *(volatile int*)&sm.gen_last_j[G % kBiasBufs] + kStages + 2 * kTmemBufs;
          }
        }
        free_buf = __shfl_sync(0xffffffffu, free_buf ? 1 : 0, 0) != 0;
        if (free_buf) {
          const float2* stp = a.stat + (int64_t)(rho0 / a.RPC) * kTile + 4 * lane;
          const float2 s0 = __ldcg(stp), s1 = __ldcg(stp + 1), s2 = __ldcg(stp + 2), s3 = __ldcg(stp + 3);
          reinterpret_cast<float4*>(sm.nbias[G % kBiasBufs])[lane] = make_float4(-s0.y, -s1.y, -s2.y, -s3.y);
          if (lane == 0) *(volatile int*)&sm.p2_rho[G % kBiasBufs] = rho0;
          __syncwarp();
          if (lane == 0) {
            __threadfence_block();
            *(volatile int*)&sm.p2_ready_gen = G;
          }
          ++G;
          // shift the window down by one and reserve a run for its new last place
          const int nrho = __shfl_down_sync(0xffffffffu, my_rho, 1);
          const bool nmine = __shfl_down_sync(0xffffffffu, mine ? 1 : 0, 1) != 0;
          my_rho = nrho, mine = nmine;
          if (lane == kBiasBufs - 1) my_rho = atomicAdd(queue + 1, 1), mine = false;
          if (lane >= kBiasBufs) my_rho = NR, mine = false;
          staged = true;
          t_progress = global_ns();
        }
      }
      if (!staged) {
        __nanosleep(100);
        if ((++it & 63) == 0) {
          bool give_up = *abort_flag != 0;
          if (!give_up && global_ns() - t_progress > a.wait_ns) {
            give_up = true;
            if (lane == 0) *abort_flag = 1, atomicCAS(a.status, 0, 13 | (G << 8));
          }
          ok = !__any_sync(0xffffffffu, give_up);
        }
      }
    }
    if (lane == 0) *(volatile int*)&sm.p2_total = G - 1;   // every reserved run that exists has been staged
  } else if (warp == 1 || warp == kMma2Warp) {
    // ================================================================= MMA issuers
    // Two threads take turns (even / odd sub-items), so that one waits and sets up while the other's
    // instructions drain into the tensor pipe.  tcgen05.commit tracks the issuing thread's own MMAs.
    if (lane == 0) {
      const uint32_t k_lo = umma_desc_lo(smem_u32(sm.k[0])), q_lo = umma_desc_lo(smem_u32(sm.q[0]));
      bool ok = true;
      int stops = 0;
      for (int j = warp == 1 ? 0 : 1; ok && stops < kTmemBufs / 2; j += 2) {
        const int stage = j % kStages, buf = j % kTmemBufs;
        ok = mbar_wait(smem_u32(&sm.full[j % kFullBars]), (j / kFullBars) & 1, abort_flag, a.status, 21 | (j << 8), a.wait_ns);
        if (!ok) break;
        const int tq = sm.desc[j % kRing].type;
        const int type = tq & 0xff;
        ok = mbar_wait(smem_u32(&sm.tmem_empty[buf]), ((j / kTmemBufs) & 1) ^ 1, abort_flag, a.status, 22 | (j << 8), a.wait_ns);
        if (!ok) break;
        if (type == kP1 || type == kP2) {
          ok = mbar_wait(smem_u32(&sm.q_full[j & 1]), (tq >> 9) & 1, abort_flag, a.status, 23 | (j << 8), a.wait_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t kd = k_lo + stage * (kTileBytes >> 4);
          const uint32_t qd = q_lo + (j & 1) * (kTileBytes >> 4);
          const uint32_t a_lo = type == kP1 ? qd : kd, b_lo = type == kP1 ? kd : qd;
          const uint32_t d = tmem_base + buf * kTile;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;
            umma_bf16(d, umma_desc_from_lo(a_lo + off), umma_desc_from_lo(b_lo + off), ks > 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&sm.empty[stage]));
          umma_commit(smem_u32(&sm.tmem_full[buf]));
        } else {
          stops += type == kStop;
          mbar_arrive(smem_u32(&sm.empty[stage]));
          mbar_arrive(smem_u32(&sm.tmem_full[buf]));
        }
      }
    }
  } else if (warp < 2 + kConsumerWarps) {
    // ================================================================= consumers
    const int group = (warp - 2) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;  // TMEM lane: query row (P1) or key within the tile (P2)
    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + group * kTile;
    const uint32_t bar_full = smem_u32(&sm.tmem_full[group]), bar_empty = smem_u32(&sm.tmem_empty[group]);
    float m_run = kMinRowMax, l_run = 0.f;
    for (int j = group;; j += kTmemBufs) {
      bool ok = mbar_wait(bar_full, (j / kTmemBufs) & 1, abort_flag, a.status, 31 | (j << 8), a.wait_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      Desc d = sm.desc[j % kRing];
      d.type &= 0xff;
      if (d.type == kStop) break;
      if (d.type == kNop) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty);
        continue;
      }
      tc_fence_after();
      const int t0 = d.tile * kTile;
      const bool tail = t0 + kTile > a.n;  // tile touches the window keys or the end of the sequence

      if (d.type == kP1) {
        // ---------------------------------------------------------- P1: running (max, sum) of this row
        if (d.first) m_run = kMinRowMax, l_run = 0.f;
        const int limit = a.n + row % W;   // last key this window row sees
        if (!kGrouped && quad * 32 >= d.n_heads * W) {
          // a short row block (the group's last heads): none of this warp's rows exists, nothing reads their pair
          // (the grouped output is only chosen when the heads fill the block)
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_empty);
        } else {
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          float v[32];
          load_logits(taddr + cc * 32, v, tail, t0 + cc * 32, limit);
          if (cc == 3) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty);
          }
          // The running sum is kept relative to a reference m_run that need not be the row maximum: any
          // reference gives the same (m, l) up to rounding as long as the sum stays inside the fp32 range.
          // So the maximum is only taken on the run's first slice, or when a sum leaves that range.
          const uint64_t scale2 = pack2(kScale, kScale);
          auto slice_sum = [&](float ref) {
            const uint64_t negm2 = pack2(-ref, -ref);
            uint64_t sum2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
            for (int jj = 0; jj < 32; jj += 2) {
              float x0, x1;
              unpack2(fma2(pack2(v[jj], v[jj + 1]), scale2, negm2), x0, x1);
              sum2[(jj >> 1) & 1] = add2(sum2[(jj >> 1) & 1], pack2(ex2(x0), ex2(x1)));
            }
            float sum[4];
            unpack2(sum2[0], sum[0], sum[1]);
            unpack2(sum2[1], sum[2], sum[3]);
            return (sum[0] + sum[1]) + (sum[2] + sum[3]);
          };
          float part = 0.f;
          bool in_range = false;
          if (!(d.first && cc == 0)) {
            part = slice_sum(m_run);
            in_range = l_run + part < 3.0e38f;   // false for infinities and NaNs too
          }
          if (!in_range) {
            float mx[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
            for (int pr = 2; pr < 16; ++pr) mx[pr & 3] = max3(mx[pr & 3], v[2 * pr], v[2 * pr + 1]);
            const float m_new = fmaxf(max3(mx[0], mx[1], mx[2]) * kScale, fmaxf(mx[3] * kScale, m_run));
            l_run *= ex2(m_run - m_new);
            m_run = m_new;
            part = slice_sum(m_run);
          }
          l_run += part;
        }
        }
        if (d.part_slot >= 0) {
          // this group's last tile of the run: publish the pair; the last warp of the chunk's
          // quadrant merges all of them in slot order
          // (the pair is normalised to a sum in [1, 2), its power of two moved into the reference, so that the
          // merge adds numbers of like size whatever the reference was)
          float m_pub = m_run, l_pub = l_run;
          if (l_run > 0.f) {
            const int bits = __float_as_int(l_run);
            m_pub = m_run + (float)((bits >> 23) - 127);
            l_pub = __int_as_float((bits & 0x007fffff) | 0x3f800000);
          }
          a.part[((int64_t)d.chunk * (a.ppr * a.RPC) + d.part_slot) * kTile + row] = make_float2(m_pub, l_pub);
          __threadfence();
          __syncwarp();
          int prev = 0;
          if (lane == 0) prev = atomicAdd(a.done + d.chunk * 4 + quad, 1);
          prev = __shfl_sync(0xffffffffu, prev, 0);
          if (prev + 1 == a.expected) {
            __threadfence();
            const float2 ml = merge_pairs(a.part + (int64_t)d.chunk * (a.ppr * a.RPC) * kTile + row, a.expected);
            a.stat[(int64_t)d.chunk * kTile + row] = make_float2(ml.x, ml.x + log2f(ml.y));
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(a.ready + d.chunk, 1);
          }
        }
      } else {
        // ---------------------------------------------------------- P2: column sums of this key
        const int t = t0 + row;
        const float* nb = sm.nbias[d.nbias_buf];
        constexpr int kHeadsPerSlice = W >= 32 ? 1 : 32 / W;  // heads inside one 32-row TMEM load
        float* out = a.csum + (int64_t)d.head0 * a.L + t;
        constexpr bool grouped = kGrouped;
        const float* hw = a.head_w + d.part_slot;
        float wv[4] = {0.f, 0.f, 0.f, 0.f};   // the block's head weights when it holds at most four heads
        if (grouped && W >= 32) {
#pragma unroll
          for (int hl = 0; hl < 128 / (W >= 32 ? W : 32); ++hl)
            if (hl < d.n_heads) wv[hl] = __ldg(hw + hl);
        }
        float head_acc = 0.f, zmax = -INFINITY, msum = 0.f;
        // a finished head: its column sum goes to memory, or into the group's weighted maximum and mass
        auto head_done = [&](int hl, float c, float w) {
          if (hl >= d.n_heads) return;
          if (!grouped) {
            if (t < a.L) out[(int64_t)hl * a.L] = c;
          } else {
            zmax = fmaxf(zmax, w * (c * a.lw_scale));
            msum += c;
          }
        };
        // a short row block has fewer slices of query rows (never with the grouped output)
        const int cc_end = kGrouped ? 4 : min(4, (d.n_heads * W + 31) / 32);
#pragma unroll 1
        for (int cc = 0; cc < cc_end; ++cc) {
          float v[32];
          tmem_ld32(taddr + cc * 32, v);
          if (cc == cc_end - 1) {  // all TMEM loads of this sub-item are done: the next tile's MMAs may run during the math
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty);
          }
          uint64_t acc2[kHeadsPerSlice];   // per head of the slice: two running sums
#pragma unroll
          for (int hh = 0; hh < kHeadsPerSlice; ++hh) acc2[hh] = pack2(0.f, 0.f);
          const uint64_t scale2 = pack2(kScale, kScale);
          // the slice's exponentials; the causal test of the window keys only exists in the copy for the tiles
          // that reach past the prefix, so that the common copy is straight-line code
          auto slice = [&](auto masked) {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const float4 b4 = reinterpret_cast<const float4*>(nb)[cc * 8 + j4];
              const uint64_t bb2[2] = {pack2(b4.x, b4.y), pack2(b4.z, b4.w)};
#pragma unroll
              for (int e2 = 0; e2 < 2; ++e2) {
                const int jj = j4 * 4 + 2 * e2;
                float x0, x1;
                unpack2(fma2(pack2(v[jj], v[jj + 1]), scale2, bb2[e2]), x0, x1);
                float p0 = ex2(x0), p1 = ex2(x1);
                if constexpr (decltype(masked)::value) {
                  if (t > a.n + (cc * 32 + jj) % W) p0 = 0.f;
                  if (t > a.n + (cc * 32 + jj + 1) % W) p1 = 0.f;
                }
                acc2[W >= 32 ? 0 : jj / W] = add2(acc2[W >= 32 ? 0 : jj / W], pack2(p0, p1));
              }
            }
          };
          if (tail) slice(std::true_type{});
          else slice(std::false_type{});
          float acc[kHeadsPerSlice][2];
#pragma unroll
          for (int hh = 0; hh < kHeadsPerSlice; ++hh) unpack2(acc2[hh], acc[hh][0], acc[hh][1]);
          if (W >= 32) {
            head_acc += acc[0][0] + acc[0][1];
            const int rows_done = (cc + 1) * 32;
            if (rows_done % W == 0) {
              const int hl = rows_done / W - 1;
              head_done(hl, head_acc, hl == 0 ? wv[0] : hl == 1 ? wv[1] : hl == 2 ? wv[2] : wv[3]);
              head_acc = 0.f;
            }
          } else {
#pragma unroll
            for (int hh = 0; hh < kHeadsPerSlice; ++hh) {
              const int hl = cc * kHeadsPerSlice + hh;
              head_done(hl, acc[hh][0] + acc[hh][1], grouped && hl < d.n_heads ? __ldg(hw + hl) : 0.f);
            }
          }
        }
        if (grouped && t < a.L) {
          const int64_t o = (int64_t)d.first * a.L + t;
          a.zgrp[o] = zmax;
          a.mgrp[o] = msum;
        }
      }
    }
  }

  // ------------------------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Rank-5 bf16 tensor map whose innermost dimension is one 64-element half of a 128-element row and
// one of whose outer dimensions selects the half (stride 128 bytes): a box that spans both halves lands
// in shared memory as two [rows][64] blocks, which is the 128-byte-swizzled K-major operand layout.
bool make_map5(CUtensorMap* map, const void* base, const cuuint64_t (&dims)[5], const cuuint64_t (&strides)[4],
               const cuuint32_t (&box)[5]) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A dimension of extent one may carry any stride; give it a legal one (in bytes).
cuuint64_t legal_stride(uint64_t extent, int64_t stride_elems, cuuint64_t fallback_bytes) {
  return (extent == 1 || stride_elems <= 0) ? fallback_bytes : (cuuint64_t)stride_elems * 2;
}

template <int W, bool kGrouped>
cudaError_t launch_wg(const CUtensorMap& qm, const CUtensorMap& km, const TcArgs& a, int grid, cudaStream_t st) {
  const size_t smem = sizeof(Smem);
  auto kernel = score_tc_kernel<W, kGrouped>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid), cfg.blockDim = dim3(kThreads), cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;  // all CTAs co-resident: CTAs wait on flags other CTAs set
  cfg.attrs = attr, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, qm, km, a);
}
template <int W>
cudaError_t launch_w(const CUtensorMap& qm, const CUtensorMap& km, const TcArgs& a, int grid, cudaStream_t st) {
  return a.zgrp ? launch_wg<W, true>(qm, km, a, grid, st) : launch_wg<W, false>(qm, km, a, grid, st);
}

}  // namespace

bool score_tc_supported(const ckv_shape& s) {
  if (s.dtype != CKV_BF16) return false;
  if (s.window != 16 && s.window != 32 && s.window != 64) return false;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  return major == 10 && encode_fn() != nullptr;
}

TcLayout tc_layout(const ckv_shape& s) {
  TcLayout t{};
  const int G = s.n_q_heads / s.n_kv_heads;
  t.RB = (G * s.window + kTile - 1) / kTile;
  t.T = (s.seq_len + kTile - 1) / kTile;
  t.C = (int64_t)s.n_units * s.n_kv_heads * t.RB;
  t.part_bytes = (size_t)t.C * (t.T + 2) * kTile * sizeof(float2);  // at most T + 1 pairs per chunk
  t.stat_bytes = (size_t)t.C * kTile * sizeof(float2);
  t.flag_bytes = ((size_t)t.C * 5 + 2) * sizeof(int);
  return t;
}

bool score_tc_groupable(const ckv_shape& s, const ckv_params& p) {
  const bool avg = p.pool_kind == CKV_POOL_AVG && p.pool_size / 2 > 0;
  return score_tc_supported(s) && tc_layout(s).RB == 1 && s.n_q_heads >= 2 * s.n_kv_heads && !avg;
}

cudaError_t launch_score_tc(const ckv_shape& s, const void* q, const void* k, float* csum, const TcGrouped* grp,
                            void* part, void* stat, int* flags, int* status, cudaStream_t st) {
  const TcLayout t = tc_layout(s);
  TcArgs a{};
  if (grp) {
    a.zgrp = grp->zgrp, a.mgrp = grp->mgrp, a.head_w = grp->head_w, a.hw_stride = grp->hw_stride;
    a.lw_scale = (float)s.seq_len / (float)s.window;
  }
  a.Nu = s.n_units, a.H = s.n_q_heads, a.Hkv = s.n_kv_heads, a.G = a.H / a.Hkv, a.L = s.seq_len, a.W = s.window;
  a.n = a.L - a.W;
  a.RB = t.RB, a.hpb = kTile / a.W, a.T = t.T, a.C = (int)t.C;
  a.run = tuning_run_tiles();
  a.RPC = (a.T + a.run - 1) / a.run;
  if (t.C * a.RPC > (int64_t)1 << 30) return cudaErrorInvalidValue;
  a.NR = a.C * a.RPC;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = sms < a.NR ? sms : a.NR;
  const int t_last = a.T - (a.RPC - 1) * a.run;
  a.ppr = a.run < 2 ? 1 : 2;
  a.expected = (a.RPC - 1) * a.ppr + (t_last < 2 ? t_last : 2);
  a.hints = tuning_l2_hints();
  const int hpb_box = a.hpb < a.H ? a.hpb : a.H;
  a.q_bytes = 2u * 64u * 2u * (uint32_t)a.W * (uint32_t)hpb_box;
  a.q_split = hpb_box * a.W < kTile;  // a short box would pack its halves closer than the operand layout wants
  a.csum = csum, a.part = (float2*)part, a.stat = (float2*)stat;
  a.done = flags, a.ready = flags + 4 * a.C, a.queue = flags + 5 * a.C, a.status = status;
  a.wait_ns = wait_limit_ns();
  CUtensorMap qm, km;
  {
    // Q: [unit][half][head][row][64]; box = one row block (hpb heads x W rows) x both halves
    const cuuint64_t row_b = legal_stride(a.W, s.q_stride_row, kHeadDim * 2);
    const cuuint64_t head_b = legal_stride(a.H, s.q_stride_head, row_b * a.W);
    const cuuint64_t unit_b = legal_stride(a.Nu, s.q_stride_unit, head_b * a.H);
    const cuuint64_t dims[5] = {64, (cuuint64_t)a.W, (cuuint64_t)a.H, 2, (cuuint64_t)a.Nu};
    const cuuint64_t strides[4] = {row_b, head_b, 128, unit_b};
    const cuuint32_t box[5] = {64, (cuuint32_t)a.W, (cuuint32_t)hpb_box, a.q_split ? 1u : 2u, 1};
    if (!make_map5(&qm, q, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    // K: [unit][head][half][token][64]; box = 128 tokens x both halves
    const cuuint64_t tok_b = legal_stride(a.L, s.kv_stride_tok, kHeadDim * 2);
    const cuuint64_t head_b = legal_stride(a.Hkv, s.kv_stride_head, tok_b * a.L);
    const cuuint64_t unit_b = legal_stride(a.Nu, s.kv_stride_unit, head_b * a.Hkv);
    const cuuint64_t dims[5] = {64, (cuuint64_t)a.L, 2, (cuuint64_t)a.Hkv, (cuuint64_t)a.Nu};
    const cuuint64_t strides[4] = {tok_b, 128, head_b, unit_b};
    const cuuint32_t box[5] = {64, kTile, 2, 1, 1};
    if (!make_map5(&km, k, dims, strides, box)) return cudaErrorInvalidValue;
  }
  cudaError_t e;   // flags: zeroed by the caller
  if (a.W == 16) e = launch_w<16>(qm, km, a, grid, st);
  else if (a.W == 32) e = launch_w<32>(qm, km, a, grid, st);
  else e = launch_w<64>(qm, km, a, grid, st);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ckv
