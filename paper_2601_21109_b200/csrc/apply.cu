// cwl_apply: adapted projection (Sec. III-F) with the boundary cross-fade (Sec. III-D).
//
//   y_t = x_t W + ((x_t A) * g_t) B,   g_t[j] = (1-lam_t) s_p [j < r_p] + lam_t s_c [j < r_c]
//
// which, by linearity, equals blending the outgoing and incoming adapter outputs.  Three launches:
//   1. shrink   P = X A at the ladder's full rank R        (tcgen05 GEMM, split along d_in, fp32 partials)
//   2. gate     H' = bf16(g * sum of partials)             (per-row rank mask, scale and cross-fade weight)
//   3. project  Y = bf16([X | H'] [W ; B])                 (tcgen05 GEMM: the K loop runs over d_in, then
//                                                           over R, into ONE TMEM accumulator)
// Both GEMMs are one persistent, warp-specialised kernel: a TMA producer warp, an MMA issuer warp
// (tcgen05.mma, cta_group::1, 128 x BN x 16, bf16 -> fp32 in TMEM) and four epilogue warps that read
// the accumulator back with tcgen05.ld.  TMEM holds two accumulators so the epilogue of one tile
// overlaps the main loop of the next.  The left operand is K-major (rows of X), the right operand
// is N-major (rows of W are contiguous in d_out), both 128-byte swizzled as TMA writes them.
//
// Every wait on an mbarrier is bounded: when it runs out the CTA raises CWL_ERR_TIMEOUT in the
// status word, drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>
#include <unordered_map>

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int BM = 128;             // rows per tile = TMEM lanes
constexpr int BK = 64;              // K elements per stage = one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int kGemmThreads = 192;   // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr int kEpilogueThreads = 128;
constexpr int kGroupM = 16;         // row tiles per raster group (keeps their X rows L2-resident)
constexpr int kNumSmsPlanned = 148; // used where the answer must not depend on the device
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

enum : int { MODE_PROJECT = 0, MODE_SHRINK = 1 };

struct GemmParams {
  int M;            // rows (tokens)
  int N;            // columns of the result
  int K0, K1;       // depth of phase 0 (d_in) and phase 1 (R, 0 when there is no adapter)
  int n_m_tiles, n_n_tiles;
  int splits;       // split-K factor over phase 0 (shrink only)
  int kb_per_split; // K blocks per split
  void* out;        // PROJECT: bf16 [M, ld_out];  SHRINK: fp32 [splits, M, ld_out]
  int64_t ld_out;
  int32_t* status_word;
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], 128 x N x 16, bf16 in, fp32 out
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrives once every MMA issued so far by this thread has finished
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout code 2), descriptor version 1.
// lbo / sbo are byte offsets: for the K-major operand sbo = distance between 8-row groups (lbo unused);
// for the N-major operand lbo = distance between 64-column atoms, sbo = distance between 8-deep K groups.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor of kind::f16: fp32 accumulate, bf16 x bf16, A K-major, B N-major.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ------------------------------------------------------------------------------------ the GEMM
template <int BN, int STAGES>
struct SmemPlan {
  static constexpr int kABytes = BM * BK * 2;       // 16 KB, one TMA box
  static constexpr int kBBytes = BN * BK * 2;       // BN/64 TMA boxes of 64 x 64
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTileBytes = STAGES * kStageBytes;
  static constexpr int kBarBytes = (2 * STAGES + 4) * 8 + 16;
  static constexpr int kTotal = kTileBytes + kBarBytes + 1024;  // + slack for 1024-byte alignment
};

struct TileCoord { int m_tile, n_tile, split; };

__device__ __forceinline__ TileCoord tile_coord(int tile, const GemmParams& p) {
  TileCoord c;
  c.split = tile % p.splits;
  tile /= p.splits;
  const int per_group = kGroupM * p.n_n_tiles;
  const int group = tile / per_group, within = tile - group * per_group;
  const int first_m = group * kGroupM;
  const int gsize = min(kGroupM, p.n_m_tiles - first_m);
  c.m_tile = first_m + within % gsize;
  c.n_tile = within / gsize;
  return c;
}

// K blocks a tile runs over: phase 0 blocks [kb0, kb1) of X/W, then all of phase 1 (H'/B)
__device__ __forceinline__ void tile_k_range(const TileCoord& c, const GemmParams& p, int& kb0, int& kb1, int& nkb1) {
  const int nkb0 = (p.K0 + BK - 1) / BK;
  kb0 = c.split * p.kb_per_split;
  kb1 = min(nkb0, kb0 + p.kb_per_split);
  nkb1 = (p.K1 + BK - 1) / BK;
}

template <int BN, int STAGES, int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a0, const __grid_constant__ CUtensorMap tm_b0,
            const __grid_constant__ CUtensorMap tm_a1, const __grid_constant__ CUtensorMap tm_b1,
            const GemmParams p) {
  using Plan = SmemPlan<BN, STAGES>;
  constexpr uint32_t kTmemCols = 2 * BN;            // two accumulators (a power of two >= 32)
  static_assert(BN % 64 == 0 && BN >= 64 && BN <= 256, "BN is a multiple of the 64-column swizzle atom");
  static_assert(kTmemCols == 128 || kTmemCols == 256 || kTmemCols == 512, "TMEM columns: power of two");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;     // swizzled tiles need 1024-byte alignment
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bars = base + Plan::kTileBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + Plan::kTileBytes + (2 * STAGES + 4) * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + Plan::kTileBytes + (2 * STAGES + 4) * 8 + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.n_m_tiles * p.n_n_tiles * p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), kEpilogueThreads); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm_a0);
    prefetch_tmap(&tm_b0);
    if (p.K1 > 0) { prefetch_tmap(&tm_a1); prefetch_tmap(&tm_b1); }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;          // running stage counter across tiles
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const TileCoord c = tile_coord(tile, p);
        int kb0, kb1, nkb1;
        tile_k_range(c, p, kb0, kb1, nkb1);
        const int n_blocks = (kb1 - kb0) + nkb1;
        for (int i = 0; i < n_blocks; ++i, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const bool phase1 = i >= (kb1 - kb0);
          const int k = phase1 ? (i - (kb1 - kb0)) * BK : (kb0 + i) * BK;
          const CUtensorMap* ma = phase1 ? &tm_a1 : &tm_a0;
          const CUtensorMap* mb = phase1 ? &tm_b1 : &tm_b0;
          const uint32_t sa = base + s * Plan::kStageBytes, sb = sa + Plan::kABytes;
          mbar_expect_tx(full_bar(s), Plan::kStageBytes);
          tma_load_2d(sa, ma, full_bar(s), k, c.m_tile * BM);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            tma_load_2d(sb + j * (BK * 128), mb, full_bar(s), c.n_tile * BN + j * 64, k);
        }
      }
      if (!ok) {
        // drain: give the copies already issued a bounded chance to land before the CTA leaves
        for (uint32_t back = 1; back <= (uint32_t)STAGES && back <= it; ++back) {
          const uint32_t j = it - back;
          unsigned long long t0 = global_timer();
          while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1u) && global_timer() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BM, BN);
      uint32_t it = 0, local_tile = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local_tile) {
        const TileCoord c = tile_coord(tile, p);
        int kb0, kb1, nkb1;
        tile_k_range(c, p, kb0, kb1, nkb1);
        const int n_blocks = (kb1 - kb0) + nkb1;
        const uint32_t acc = local_tile & 1u, acc_ph = (local_tile >> 1) & 1u;
        if (!mbar_wait(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int i = 0; i < n_blocks; ++i, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const bool phase1 = i >= (kb1 - kb0);
          const int k = phase1 ? (i - (kb1 - kb0)) * BK : (kb0 + i) * BK;
          const int k_left = (phase1 ? p.K1 : p.K0) - k;         // multiple of 16
          const int k_steps = k_left >= BK ? BK / UMMA_K : k_left / UMMA_K;
          const uint32_t sa = base + s * Plan::kStageBytes, sb = sa + Plan::kABytes;
          for (int kk = 0; kk < k_steps; ++kk) {
            const uint64_t da = make_smem_desc(sa + kk * (UMMA_K * 2), 16, 1024);
            const uint64_t db = make_smem_desc(sb + kk * (UMMA_K * 128), BK * 128, 1024);
            umma_bf16(d_tmem, da, db, idesc, (i | kk) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(s));            // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(acc_full_bar(acc)); // accumulator complete
      }
      if (!ok) {
        // give the MMAs still in flight a bounded time to retire before TMEM is released
        unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 1000000ull) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int lane_group = warp & 3;              // TMEM lanes this warp may read: 32*lane_group ..
    const int row_in_tile = lane_group * 32 + lane;
    uint32_t local_tile = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local_tile) {
      const TileCoord c = tile_coord(tile, p);
      const uint32_t acc = local_tile & 1u, acc_ph = (local_tile >> 1) & 1u;
      if (!mbar_wait(acc_full_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row = c.m_tile * BM + row_in_tile;
      const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(lane_group * 32) << 16);
#pragma unroll 1
      for (int cc = 0; cc < BN / 32; ++cc) {
        const int col = c.n_tile * BN + cc * 32;
        if (col >= p.N) break;                     // warp-uniform
        uint32_t v[32];
        tmem_ld32(t_row + cc * 32, v);
        tmem_ld_wait();
        if (row < p.M) {
          if (MODE == MODE_PROJECT) {
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)row * p.ld_out + col;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (col + g * 8 < p.N) {             // N is a multiple of 8: a granule is all in or all out
                uint4 q;
                q.x = pack_bf16(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
                q.y = pack_bf16(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
                q.z = pack_bf16(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
                q.w = pack_bf16(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
                *reinterpret_cast<uint4*>(out + g * 8) = q;
              }
            }
          } else {
            float* out = reinterpret_cast<float*>(p.out) + ((int64_t)c.split * p.M + row) * p.ld_out + col;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              if (col + g * 4 < p.N) {
                uint4 q = make_uint4(v[g * 4 + 0], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
                *reinterpret_cast<uint4*>(out + g * 4) = q;
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty_bar(acc));
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) flag_status(p.status_word, CWL_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// --------------------------------------------------------------------------------------- gate
// H'[t, j] = bf16(g_t[j] * sum_s partial[s][t][j]).  Each block expands the chunk table into one
// row descriptor per token in shared memory, then all threads apply it.
constexpr int kGateRows = 32;
constexpr int kGateThreads = 256;

struct RowGate { float w_in, w_out; int r_in, r_out; };  // g[j] = w_in [j < r_in] + w_out [j < r_out]

__global__ void __launch_bounds__(kGateThreads)
gate_kernel(const float* __restrict__ partial, int splits, int T, int R, cwl_chunk_table table, int window,
            __nv_bfloat16* __restrict__ Hg) {
  __shared__ RowGate gates[kGateRows];
  const int row0 = blockIdx.x * kGateRows;
  if (threadIdx.x < kGateRows) {
    const int t = row0 + threadIdx.x;
    RowGate g{0.f, 0.f, 0, 0};
    const int C = min(*table.n_chunks, table.capacity);
    if (t < T && C > 0 && t >= table.offsets[0] && t < table.offsets[C]) {
      int lo = 0, hi = C;                          // offsets[lo] <= t < offsets[hi]
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (table.offsets[mid] <= t) lo = mid; else hi = mid;
      }
      const int c = lo, j = t - table.offsets[c];
      float lam = 1.f;
      if (c > 0 && !(table.flags[c] & 1) && j < window) lam = (float)(j + 1) / (float)(window + 1);
      g.r_in = min(max(table.rank[c], 0), R);
      g.w_in = lam * table.scale[c];
      if (lam < 1.f) {
        g.r_out = min(max(table.rank[c - 1], 0), R);
        g.w_out = (1.f - lam) * table.scale[c - 1];
      }
    }
    gates[threadIdx.x] = g;
  }
  __syncthreads();
  const int groups_per_row = R >> 2;               // 4 columns per thread step
  const int64_t split_stride = (int64_t)T * R;
  for (int idx = threadIdx.x; idx < kGateRows * groups_per_row; idx += kGateThreads) {
    const int r = idx / groups_per_row, j0 = (idx - r * groups_per_row) << 2;
    const int t = row0 + r;
    if (t >= T) break;
    const RowGate g = gates[r];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* src = partial + (int64_t)t * R + j0;
    for (int s = 0; s < splits; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(src + s * split_stride);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    auto gate = [&](int j) { return (j < g.r_in ? g.w_in : 0.f) + (j < g.r_out ? g.w_out : 0.f); };
    uint2 o;
    o.x = pack_bf16(acc.x * gate(j0), acc.y * gate(j0 + 1));
    o.y = pack_bf16(acc.z * gate(j0 + 2), acc.w * gate(j0 + 3));
    *reinterpret_cast<uint2*>(Hg + (int64_t)t * R + j0) = o;
  }
}

// ------------------------------------------------------------------------------- host: TMA maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

struct MapKey {
  const void* ptr; uint64_t inner, outer, ld; uint32_t box_inner, box_outer;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && inner == o.inner && outer == o.outer && ld == o.ld && box_inner == o.box_inner &&
           box_outer == o.box_outer;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = reinterpret_cast<size_t>(k.ptr);
    for (uint64_t v : {k.inner, k.outer, k.ld, (uint64_t)k.box_inner, (uint64_t)k.box_outer})
      h = h * 0x9E3779B97F4A7C15ull + v;
    return h;
  }
};

// bf16 row-major [outer, inner] with row stride ld (elements), box = box_inner x box_outer, 128B swizzle.
// Rows and columns outside the tensor read as zero.  Descriptors depend only on the key: cached.
bool make_map(CUtensorMap* out, const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld,
              uint32_t box_inner, uint32_t box_outer) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  const MapKey key{ptr, inner, outer, ld, box_inner, box_outer};
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
  }
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (cache.size() > 4096) cache.clear();
  cache.emplace(key, *out);
  return true;
}

int sm_count() {
  static int n = []() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return kNumSmsPlanned;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return kNumSmsPlanned;
    return v;
  }();
  return n;
}

template <int BN, int STAGES, int MODE>
cwl_status launch_gemm(const CUtensorMap& a0, const CUtensorMap& b0, const CUtensorMap& a1, const CUtensorMap& b1,
                       const GemmParams& p, cudaStream_t stream) {
  using Plan = SmemPlan<BN, STAGES>;
  auto kernel = gemm_kernel<BN, STAGES, MODE>;
  static bool configured[64] = {};  // per device; benign race: the attribute call is idempotent
  int dev = 0;
  CWL_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    CWL_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan::kTotal));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const int total = p.n_m_tiles * p.n_n_tiles * p.splits;
  const int grid = total < sm_count() ? total : sm_count();
  kernel<<<grid, kGemmThreads, Plan::kTotal, stream>>>(a0, b0, a1, b1, p);
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
}

// split-K factor of the shrink GEMM: enough CTAs to pull X at full HBM rate when T is small
int shrink_splits(int T, int d_in) {
  const int n_m = ceil_div(T, BM), nkb = ceil_div(d_in, BK);
  int s = ceil_div(kNumSmsPlanned, n_m);
  if (s > nkb) s = nkb;
  if (s > 32) s = 32;
  if (s < 1) s = 1;
  const int per = ceil_div(nkb, s);
  return ceil_div(nkb, per);        // no empty split
}

struct ApplyWorkspace { __nv_bfloat16* Hg; float* partial; };

size_t carve_apply(ApplyWorkspace& w, char* base, int T, int d_in, int R) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  size_t off = 0;
  w.Hg = reinterpret_cast<__nv_bfloat16*>(base ? base + off : nullptr);
  off = up(off + (size_t)T * R * sizeof(__nv_bfloat16));
  w.partial = reinterpret_cast<float*>(base ? base + off : nullptr);
  off = up(off + (size_t)shrink_splits(T, d_in) * T * R * sizeof(float));
  return off;
}

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_apply_workspace_bytes(int32_t T, int32_t d_in, int32_t d_out, int32_t R) {
  (void)d_out;
  if (T <= 0 || d_in <= 0 || R <= 0) return 256;
  cwl::ApplyWorkspace w;
  return cwl::carve_apply(w, nullptr, T, d_in, R);
}

extern "C" cwl_status cwl_apply(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                const void* A, int64_t lda, const void* B, int64_t ldb,
                                int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                cwl_chunk_table table, int32_t window,
                                void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                int32_t* status_word, void* stream_) {
  using namespace cwl;
  if (T < 0 || d_in < 1 || d_out < 1 || R < 0 || window < 0) return CWL_ERR_INVALID_ARG;
  if (T > 0 && (X == nullptr || Y == nullptr)) return CWL_ERR_INVALID_ARG;
  if (W == nullptr) return CWL_ERR_INVALID_ARG;
  const bool adapter = (A != nullptr && B != nullptr && R > 0);
  if (d_in % 16 != 0 || d_out % 16 != 0) return CWL_ERR_UNSUPPORTED;
  if (adapter && (R % 16 != 0 || R > CWL_MAX_RANK)) return CWL_ERR_UNSUPPORTED;
  if (ldx < d_in || ldw < d_out || ldy < d_out || (adapter && (lda < R || ldb < d_out))) return CWL_ERR_SHAPE;
  if (ldx % 8 != 0 || ldw % 8 != 0 || ldy % 8 != 0 || (adapter && (lda % 8 != 0 || ldb % 8 != 0))) return CWL_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || (adapter && (!aligned16(A) || !aligned16(B))))
    return CWL_ERR_SHAPE;
  if (T == 0) return CWL_OK;
  if (adapter && (table.offsets == nullptr || table.rank == nullptr || table.scale == nullptr ||
                  table.flags == nullptr || table.n_chunks == nullptr || table.capacity < 0))
    return CWL_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);

  ApplyWorkspace ws{nullptr, nullptr};
  if (adapter) {
    const size_t need = carve_apply(ws, static_cast<char*>(workspace), T, d_in, R);
    if (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
      return CWL_ERR_WORKSPACE;
  }

  CUtensorMap mX, mW, mH, mB, mA;
  if (!make_map(&mX, X, (uint64_t)d_in, (uint64_t)T, (uint64_t)ldx, BK, BM)) return CWL_ERR_CUDA;
  if (!make_map(&mW, W, (uint64_t)d_out, (uint64_t)d_in, (uint64_t)ldw, 64, BK)) return CWL_ERR_CUDA;

  if (adapter) {
    if (!make_map(&mA, A, (uint64_t)R, (uint64_t)d_in, (uint64_t)lda, 64, BK)) return CWL_ERR_CUDA;
    if (!make_map(&mH, ws.Hg, (uint64_t)R, (uint64_t)T, (uint64_t)R, BK, BM)) return CWL_ERR_CUDA;
    if (!make_map(&mB, B, (uint64_t)d_out, (uint64_t)R, (uint64_t)ldb, 64, BK)) return CWL_ERR_CUDA;

    // 1. shrink: partial[s] = X[:, split s of d_in] A[split s, :]
    GemmParams sp{};
    sp.M = T; sp.N = R; sp.K0 = d_in; sp.K1 = 0;
    sp.n_m_tiles = ceil_div(T, BM); sp.n_n_tiles = 1;
    sp.splits = shrink_splits(T, d_in);
    sp.kb_per_split = ceil_div(ceil_div(d_in, BK), sp.splits);
    sp.out = ws.partial; sp.ld_out = R; sp.status_word = status_word;
    cwl_status st;
    if (R <= 64)       st = launch_gemm<64, 6, MODE_SHRINK>(mX, mA, mX, mA, sp, stream);
    else if (R <= 128) st = launch_gemm<128, 6, MODE_SHRINK>(mX, mA, mX, mA, sp, stream);
    else               st = launch_gemm<256, 4, MODE_SHRINK>(mX, mA, mX, mA, sp, stream);
    if (st != CWL_OK) return st;

    // 2. gate
    gate_kernel<<<ceil_div(T, kGateRows), kGateThreads, 0, stream>>>(ws.partial, sp.splits, T, R, table, window, ws.Hg);
    CWL_CUDA_TRY(cudaGetLastError());
  }

  // 3. project: Y = [X | H'] [W ; B]
  GemmParams gp{};
  gp.M = T; gp.N = d_out; gp.K0 = d_in; gp.K1 = adapter ? R : 0;
  gp.n_m_tiles = ceil_div(T, BM); gp.n_n_tiles = ceil_div(d_out, 256);
  gp.splits = 1; gp.kb_per_split = ceil_div(d_in, BK);
  gp.out = Y; gp.ld_out = ldy; gp.status_word = status_word;
  if (adapter) return launch_gemm<256, 4, MODE_PROJECT>(mX, mW, mH, mB, gp, stream);
  return launch_gemm<256, 4, MODE_PROJECT>(mX, mW, mX, mW, gp, stream);
}

// ------------------------------------------------------------------------------ no-allocation variant
// Scratch for cwl_apply_noalloc lives in the library image itself, so a caller that may not allocate
// device memory (no cudaMalloc in its context, or an allocator it does not own) can still run the
// adapted projection.  Every device that loads the library carries this array until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CWL_NOALLOC_SCRATCH_BYTES];

namespace cwl {
namespace {

// Device address of g_noalloc_scratch on the current device.  The array's name is only a host-side
// handle here; the address the kernels need comes from cudaGetSymbolAddress, once per device.
cwl_status noalloc_scratch(void** out) {
  static std::mutex mu;
  static void* ptr_of_device[64] = {};
  int dev = 0;
  CWL_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CWL_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  if (ptr_of_device[dev] == nullptr) {
    void* p = nullptr;
    CWL_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (p == nullptr) return CWL_ERR_CUDA;
    ptr_of_device[dev] = p;
  }
  *out = ptr_of_device[dev];
  return CWL_OK;
}

}  // namespace
}  // namespace cwl

extern "C" cwl_status cwl_apply_noalloc(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                        const void* A, int64_t lda, const void* B, int64_t ldb,
                                        int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                        cwl_chunk_table table, int32_t window,
                                        void* Y, int64_t ldy, int32_t* status_word, void* stream) {
  if (T < 0 || d_in < 1 || d_out < 1 || R < 0) return CWL_ERR_INVALID_ARG;
  const bool adapter = (A != nullptr && B != nullptr && R > 0);
  if (adapter && T > 0 && cwl_apply_workspace_bytes(T, d_in, d_out, R) > (size_t)CWL_NOALLOC_SCRATCH_BYTES)
    return CWL_ERR_WORKSPACE;  // the problem needs more scratch than the built-in array holds
  void* scratch = nullptr;
  const cwl_status st = cwl::noalloc_scratch(&scratch);
  if (st != CWL_OK) return st;
  return cwl_apply(X, ldx, W, ldw, A, lda, B, ldb, T, d_in, d_out, R, table, window, Y, ldy, scratch,
                   (size_t)CWL_NOALLOC_SCRATCH_BYTES, status_word, stream);
}
