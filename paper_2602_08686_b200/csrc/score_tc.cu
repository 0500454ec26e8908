// Tensor-core window-score scan for bf16 inputs on sm_100a (Sec. 3 softmax; Eq. 4 window mass).
//
// One persistent, warp-specialised kernel does both passes over K:
//   P1 (row statistics)  D[row, key]  = Q_blk . K_tile^T   (UMMA M = 128 query rows, N = 128 keys):
//        one TMEM lane per query row, so the running row maximum and the sum of exponentials are
//        thread-local; per-run partial pairs go to global memory and the last warp to finish a chunk
//        merges them in a fixed order into (max, max + log2 sum).
//   P2 (column sums)     D[key, row]  = K_tile . Q_blk^T   (the same shared-memory tiles, operands
//        swapped): one TMEM lane per key, so c_h[t] = sum_i 2^(x[i,t] - bias_i) is thread-local.
// A "chunk" is one (unit, KV head, block of 128 query rows); a "run" is up to four consecutive key
// tiles of a chunk.  CTA b handles P1 runs b, b+grid, ... and, interleaved, the P2 runs that trail
// them by a fixed lag, so the second read of a K tile comes from L2 while its chunk's statistics are
// long complete.  K and Q tiles arrive by TMA (128-byte swizzle) and feed tcgen05.mma directly; the
// accumulators live in TMEM (four 128-column buffers) and are read back with tcgen05.ld.
//
// Every wait is bounded: an mbarrier or flag wait that exceeds its time limit records
// CKV_ERR_TIMEOUT in the work space's status word and the CTA winds down (frees TMEM, returns).
#include <cuda.h>
#include <cuda_bf16.h>

#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kTile = 128;        // keys per tile, also query rows per block
constexpr int kStages = 4;        // K-tile ring
constexpr int kTmemBufs = 4;      // accumulator buffers of 128 columns
constexpr int kRun = 4;           // key tiles per run
constexpr int kBiasSlots = 8;     // >= kStages + kTmemBufs
constexpr int kConsumerWarps = 8; // two sets of four (one warp per TMEM lane quadrant)
constexpr int kThreads = 32 * (2 + kConsumerWarps);
constexpr uint32_t kHalfBytes = 128 * 128;          // 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfBytes;     // 128 rows x 128 bf16
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// x = (q.k) * log2(e) / sqrt(128)
constexpr float kScale = 0.12751743074602467f;

// UMMA instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

struct TcArgs {
  int Nu, H, Hkv, G, L, W, n;
  int RB, hpb;          // row blocks per KV group; query heads per row block (128 / W)
  int T, RPC, C;        // key tiles per chunk; runs per chunk; chunks
  int NR, DR;           // runs in total; lag of the P2 stream behind the P1 stream, in runs
  int expected;         // partial flushes per (chunk, lane quadrant)
  uint32_t q_half_bytes;
  float* csum;
  float2* part;         // [C][2*RPC][128]
  float2* stat;         // [C][128]
  int* done;            // [C][4]
  int* ready;           // [C]
  int* status;
};

struct SubItem {
  int type;  // 0 = P1, 1 = P2
  int chunk, tile, k, tr, run_in_chunk;
};

// The fixed sequence of sub-items of one CTA; every warp role walks it independently.
struct Sched {
  int b, grid, m, phase, k;
  __device__ Sched(int b_, int grid_) : b(b_), grid(grid_), m(0), phase(0), k(0) {}
  __device__ bool next(const TcArgs& a, SubItem& s) {
    while (true) {
      const int rho1 = b + m * grid;
      if (phase == 0 && rho1 - a.DR >= a.NR) return false;
      const int rho = phase == 0 ? rho1 : rho1 - a.DR;
      if (rho >= 0 && rho < a.NR) {
        const int chunk = rho / a.RPC, ric = rho - chunk * a.RPC;
        const int tr = min(kRun, a.T - ric * kRun);
        if (k < tr) {
          s.type = phase, s.chunk = chunk, s.run_in_chunk = ric, s.tr = tr, s.k = k, s.tile = ric * kRun + k;
          ++k;
          return true;
        }
      }
      k = 0;
      if (phase == 0) {
        phase = 1;
      } else {
        phase = 0;
        ++m;
      }
    }
  }
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
                                            int code) {
  const unsigned long long t0 = global_ns();
  for (int it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255) == 255) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          int code) {
  for (int it = 0; it < 64; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, code);
}

__device__ __forceinline__ void tma_load_4d(const CUtensorMap* map, uint32_t dst, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart, groups of
// eight rows 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fff);
  d |= (uint64_t)1 << 16;               // leading byte offset (unused for swizzled K-major), canonical value 1
  d |= (uint64_t)(1024 >> 4) << 32;     // stride byte offset
  d |= (uint64_t)1 << 46;               // descriptor version
  d |= (uint64_t)2 << 61;               // SWIZZLE_128B
  return d;
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

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// ------------------------------------------------------------------------------------ shared memory
struct __align__(1024) Smem {
  uint8_t k[kStages][kTileBytes];  // K tiles: two 64-column halves of [128 rows][128 bytes], swizzled
  uint8_t q[2][kTileBytes];        // query rows of the P1 stream's chunk and of the P2 stream's chunk
  float bias[kBiasSlots][kTile];   // row biases (max + log2 sum) of the P2 tile in flight
  uint64_t full[kStages], empty[kStages], tmem_full[kTmemBufs], tmem_empty[kTmemBufs];
  uint32_t tmem_base;
  int abort_flag;
};

template <int W>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map, TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sm.full[s]), 1);
      mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    for (int b = 0; b < kTmemBufs; ++b) {
      mbar_init(smem_u32(&sm.tmem_full[b]), 1);
      mbar_init(smem_u32(&sm.tmem_empty[b]), 4);
    }
    sm.abort_flag = 0;
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

  Sched sched(blockIdx.x, gridDim.x);
  SubItem s;
  int j = 0;

  if (warp == 0) {
    // ================================================================= TMA producer
    int q_chunk[2] = {-1, -1}, q_last[2] = {-1000, -1000};
    float4 bias_reg = make_float4(0.f, 0.f, 0.f, 0.f);
    bool ok = true;
    while (ok && sched.next(a, s)) {
      const int stage = j % kStages;
      const bool reload = s.chunk != q_chunk[s.type];
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&sm.empty[stage]), ((j / kStages) & 1) ^ 1, abort_flag, a.status, 11);
        if (ok && reload) {
          const int jl = q_last[s.type];
          if (jl >= 0 && j - jl < kStages)  // the MMAs that read the old rows must have completed
            ok = mbar_wait(smem_u32(&sm.empty[jl % kStages]), (jl / kStages) & 1, abort_flag, a.status, 12);
          if (ok && s.type == 1) {  // the chunk's row statistics must be final
            const unsigned long long t0 = global_ns();
            int it = 0;
            while (ld_acquire(a.ready + s.chunk) < 4) {
              __nanosleep(64);
              if ((++it & 63) == 0) {
                if (*abort_flag) {
                  ok = false;
                  break;
                }
                if (global_ns() - t0 > kWaitLimitNs) {
                  *abort_flag = 1;
                  atomicCAS(a.status, 0, 13);
                  ok = false;
                  break;
                }
              }
            }
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      if (s.type == 1) {
        if (reload) {
          const float2* st = a.stat + (int64_t)s.chunk * kTile + 4 * lane;
          const float2 s0 = __ldcg(st), s1 = __ldcg(st + 1), s2 = __ldcg(st + 2), s3 = __ldcg(st + 3);
          bias_reg = make_float4(s0.y, s1.y, s2.y, s3.y);
        }
        reinterpret_cast<float4*>(sm.bias[j % kBiasSlots])[lane] = bias_reg;
        __syncwarp();
      }
      if (lane == 0) {
        const int g_rb = s.chunk % (a.Hkv * a.RB);
        const int u = s.chunk / (a.Hkv * a.RB), g = g_rb / a.RB, rb = g_rb % a.RB;
        const uint32_t bar = smem_u32(&sm.full[stage]);
        mbar_arrive_expect_tx(bar, kTileBytes + (reload ? 2 * a.q_half_bytes : 0));
        if (reload) {
          const uint32_t qdst = smem_u32(sm.q[s.type]);
          const int head0 = g * a.G + rb * a.hpb;
          tma_load_4d(&q_map, qdst, bar, 0, 0, head0, u);
          tma_load_4d(&q_map, qdst + kHalfBytes, bar, 64, 0, head0, u);
        }
        const uint32_t kdst = smem_u32(sm.k[stage]);
        tma_load_4d(&k_map, kdst, bar, 0, s.tile * kTile, g, u);
        tma_load_4d(&k_map, kdst + kHalfBytes, bar, 64, s.tile * kTile, g, u);
      }
      q_chunk[s.type] = s.chunk;
      q_last[s.type] = j;
      ++j;
    }
    if (!ok && lane == 0) {
      // give copies in flight time to land before the CTA's shared memory goes away
      for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ================================================================= MMA issuer
    bool ok = true;
    while (ok && sched.next(a, s)) {
      const int stage = j % kStages, buf = j % kTmemBufs;
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&sm.full[stage]), (j / kStages) & 1, abort_flag, a.status, 21) &&
             mbar_wait(smem_u32(&sm.tmem_empty[buf]), ((j / kTmemBufs) & 1) ^ 1, abort_flag, a.status, 22);
        if (ok) {
          tc_fence_after();
          const uint32_t kaddr = smem_u32(sm.k[stage]), qaddr = smem_u32(sm.q[s.type]);
          const uint32_t a_addr = s.type == 0 ? qaddr : kaddr, b_addr = s.type == 0 ? kaddr : qaddr;
          const uint32_t d = tmem_base + buf * kTile;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
            umma_bf16(d, umma_desc(a_addr + off), umma_desc(b_addr + off), ks > 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&sm.empty[stage]));
          umma_commit(smem_u32(&sm.tmem_full[buf]));
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      ++j;
    }
  } else {
    // ================================================================= consumers
    const int cw = warp - 2, set = cw >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;  // TMEM lane: query row (P1) or key within the tile (P2)
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    while (ok && sched.next(a, s)) {
      if ((j & 1) != set) {
        ++j;
        continue;
      }
      const int buf = j % kTmemBufs;
      ok = mbar_wait(smem_u32(&sm.tmem_full[buf]), (j / kTmemBufs) & 1, abort_flag, a.status, 31);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kTile;
      const int t0 = s.tile * kTile;
      const bool tail = t0 + kTile > a.n;  // tile touches the window keys or the end of the sequence

      if (s.type == 0) {
        // ---------------------------------------------------------- P1: running (max, sum) of this row
        if (s.k < 2) m_run = -INFINITY, l_run = 0.f;
        const int i = row % W;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          float v[32];
          tmem_ld32(taddr + cc * 32, v);
          if (cc == 3) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.tmem_empty[buf]));
          }
          if (tail) {
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) {
              const int t = t0 + cc * 32 + jj;
              if (t >= a.L || t > a.n + i) v[jj] = -INFINITY;
            }
          }
          float cmax = v[0];
#pragma unroll
          for (int jj = 1; jj < 32; ++jj) cmax = fmaxf(cmax, v[jj]);
          const float m_new = fmaxf(m_run, cmax * kScale);
          if (m_new != -INFINITY) {
            float acc = 0.f;
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) acc += ex2(fmaf(v[jj], kScale, -m_new));
            l_run = l_run * ex2(m_run - m_new) + acc;
            m_run = m_new;
          }
        }
        if (s.k + 2 >= s.tr) {
          // this warp's last tile of the run: publish the partial pair; the last warp of the chunk's
          // quadrant merges all of them in slot order
          const int slot = s.run_in_chunk * 2 + (s.k & 1);
          a.part[((int64_t)s.chunk * (2 * a.RPC) + slot) * kTile + row] = make_float2(m_run, l_run);
          __threadfence();
          __syncwarp();
          int prev = 0;
          if (lane == 0) prev = atomicAdd(a.done + s.chunk * 4 + quad, 1);
          prev = __shfl_sync(0xffffffffu, prev, 0);
          if (prev + 1 == a.expected) {
            __threadfence();
            const float2* p = a.part + (int64_t)s.chunk * (2 * a.RPC) * kTile + row;
            float m = -INFINITY;
            for (int sl = 0; sl < a.expected; ++sl) m = fmaxf(m, __ldcg(p + (int64_t)sl * kTile).x);
            float l = 0.f;
            for (int sl = 0; sl < a.expected; ++sl) {
              const float2 pr = __ldcg(p + (int64_t)sl * kTile);
              if (pr.y > 0.f) l += pr.y * ex2(pr.x - m);
            }
            a.stat[(int64_t)s.chunk * kTile + row] = make_float2(m, m + log2f(l));
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(a.ready + s.chunk, 1);
          }
        }
      } else {
        // ---------------------------------------------------------- P2: column sums of this key
        const int t = t0 + row;
        const float* bias = sm.bias[j % kBiasSlots];
        const int g_rb = s.chunk % (a.Hkv * a.RB);
        const int u = s.chunk / (a.Hkv * a.RB), g = g_rb / a.RB, rb = g_rb % a.RB;
        constexpr int kHeadsPerChunk = W >= 32 ? 1 : 32 / W;  // heads inside one 32-row TMEM load
        float head_acc = 0.f;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          float v[32];
          tmem_ld32(taddr + cc * 32, v);
          float acc[kHeadsPerChunk];
#pragma unroll
          for (int hh = 0; hh < kHeadsPerChunk; ++hh) acc[hh] = 0.f;
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) {
            const float4 b4 = reinterpret_cast<const float4*>(bias)[cc * 8 + j4];
            const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int jj = j4 * 4 + e;
              float p = ex2(fmaf(v[jj], kScale, -bb[e]));
              if (tail) {
                const int i = (cc * 32 + jj) % W;
                if (t > a.n + i) p = 0.f;
              }
              acc[W >= 32 ? 0 : jj / W] += p;
            }
          }
          if (cc == 3) {  // all bias reads and TMEM loads of this sub-item are done
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.tmem_empty[buf]));
          }
          if (W >= 32) {
            head_acc += acc[0];
            const int rows_done = (cc + 1) * 32;
            if (rows_done % W == 0) {
              const int hl = rb * a.hpb + rows_done / W - 1;
              if (hl < a.G && t < a.L) a.csum[((int64_t)u * a.H + g * a.G + hl) * a.L + t] = head_acc;
              head_acc = 0.f;
            }
          } else {
#pragma unroll
            for (int hh = 0; hh < kHeadsPerChunk; ++hh) {
              const int hl = rb * a.hpb + cc * kHeadsPerChunk + hh;
              if (hl < a.G && t < a.L) a.csum[((int64_t)u * a.H + g * a.G + hl) * a.L + t] = acc[hh];
            }
          }
        }
      }
      ++j;
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

// bf16 tensor [d3][d2][d1][128] with element strides (s1, s2, s3); box [1][b2][b1][64], 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, uint64_t d1, uint64_t d2, uint64_t d3, int64_t s1, int64_t s2,
              int64_t s3, uint32_t b1, uint32_t b2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  // a dimension of extent one may carry any stride; give it a legal one
  if (d1 == 1 || s1 <= 0) s1 = kHeadDim;
  if (d2 == 1 || s2 <= 0) s2 = s1 * (int64_t)d1;
  if (d3 == 1 || s3 <= 0) s3 = s2 * (int64_t)d2;
  const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, d1, d2, d3};
  const cuuint64_t strides[3] = {(cuuint64_t)s1 * 2, (cuuint64_t)s2 * 2, (cuuint64_t)s3 * 2};
  const cuuint32_t box[4] = {64, b1, b2, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int W>
cudaError_t launch_w(const CUtensorMap& qm, const CUtensorMap& km, const TcArgs& a, int grid, cudaStream_t st) {
  const size_t smem = sizeof(Smem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<W>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid), cfg.blockDim = dim3(kThreads), cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;  // all CTAs co-resident: CTAs wait on flags other CTAs set
  cfg.attrs = attr, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, score_tc_kernel<W>, qm, km, a);
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
  t.RPC = (t.T + kRun - 1) / kRun;
  t.C = (int64_t)s.n_units * s.n_kv_heads * t.RB;
  t.part_bytes = (size_t)t.C * 2 * t.RPC * kTile * sizeof(float2);
  t.stat_bytes = (size_t)t.C * kTile * sizeof(float2);
  t.flag_bytes = (size_t)t.C * 5 * sizeof(int);
  return t;
}

cudaError_t launch_score_tc(const ckv_shape& s, const void* q, const void* k, float* csum, void* part, void* stat,
                            int* flags, int* status, cudaStream_t st) {
  const TcLayout t = tc_layout(s);
  if (t.C > (int64_t)1 << 24) return cudaErrorInvalidValue;
  TcArgs a{};
  a.Nu = s.n_units, a.H = s.n_q_heads, a.Hkv = s.n_kv_heads, a.G = a.H / a.Hkv, a.L = s.seq_len, a.W = s.window;
  a.n = a.L - a.W;
  a.RB = t.RB, a.hpb = kTile / a.W, a.T = t.T, a.RPC = t.RPC, a.C = (int)t.C;
  a.NR = a.C * a.RPC;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = sms < a.NR ? sms : a.NR;
  a.DR = a.RPC + 2 * grid;
  const int t_last = a.T - (a.RPC - 1) * kRun;
  a.expected = 2 * (a.RPC - 1) + (t_last < 2 ? t_last : 2);
  const int hpb_box = a.hpb < a.H ? a.hpb : a.H;
  a.q_half_bytes = 64u * 2u * (uint32_t)a.W * (uint32_t)hpb_box;
  a.csum = csum, a.part = (float2*)part, a.stat = (float2*)stat;
  a.done = flags, a.ready = flags + 4 * a.C, a.status = status;
  CUtensorMap qm, km;
  if (!make_map(&qm, q, a.W, a.H, a.Nu, s.q_stride_row, s.q_stride_head, s.q_stride_unit, a.W, hpb_box) ||
      !make_map(&km, k, a.L, a.Hkv, a.Nu, s.kv_stride_tok, s.kv_stride_head, s.kv_stride_unit, kTile, 1))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaMemsetAsync(flags, 0, t.flag_bytes, st);
  if (e != cudaSuccess) return e;
  if (a.W == 16) e = launch_w<16>(qm, km, a, grid, st);
  else if (a.W == 32) e = launch_w<32>(qm, km, a, grid, st);
  else e = launch_w<64>(qm, km, a, grid, st);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ckv
