// cwl_apply: adapted projection (Sec. III-F) with the boundary cross-fade (Sec. III-D).
//
//   y_t = x_t W + ((x_t A) * g_t) B,   g_t[j] = (1-lam_t) s_p [j < r_p] + lam_t s_c [j < r_c]
//
// which, by linearity, equals blending the outgoing and incoming adapter outputs.  ONE persistent,
// warp-specialised kernel does all of it, launched as clusters of two CTAs: a pair owns 256 rows and
// issues tcgen05.mma with cta_group::2, so each CTA stages only its 128 rows of the left operand and
// HALF of the right operand per pipeline step (a third less shared-memory fill per FLOP than a
// single-CTA 128 x 256 tile, which is what bounded the single-CTA version).
// Each pair first works through its share of SHRINK items
//   P[split] = X[:, split of d_in] A[split, :]   (full ladder rank R, fp32 partials when d_in is split),
// the CTA that completes a row tile's last split sums the partials, applies the per-row gate (rank
// mask, scale and cross-fade weight from the chunk table, expanded per row in shared memory) and
// publishes H' = bf16(g * X A) with a release flag; then the CTAs work through the PROJECT tiles
//   Y = bf16([X | H'] [W ; B])
// whose K loop runs over d_in and then over R into ONE TMEM accumulator (the TMA producer acquires the
// row tile's flag before its first H' load, ~d_in/64 pipeline steps after the tile began).
//
// Roles per CTA: warp 0 = TMA producer (cp.async.bulk.tensor, 128-byte swizzle, bytes counted on the
// leader's mbarrier), warp 1 = tcgen05.mma issuer in the leader CTA only (256 x N x 16 across the pair,
// bf16 -> fp32 in TMEM; tcgen05.commit multicast frees the stage in both CTAs), warps 2..5 = epilogue
// (tcgen05.ld of the CTA's own 128 accumulator rows).  TMEM holds two accumulators so the epilogue of
// one item overlaps the main loop of the next.  The left operand
// is K-major (rows of X / H'), the right operand is N-major (rows of W, A, B are contiguous in their
// output dimension), exactly as the matrices sit in HBM.
//
// Every wait (mbarrier or flag) is bounded: when it runs out the CTA raises CWL_ERR_TIMEOUT in the
// status word, drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <unordered_map>

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int BM = 128;             // rows per tile = TMEM lanes
constexpr int BN = 256;             // columns per projection tile = one TMEM accumulator
constexpr int BK = 64;              // K elements per stage = one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
#ifndef CWL_STAGES
#define CWL_STAGES 6
#endif
constexpr int kStages = CWL_STAGES;
constexpr int kGemmThreads = 192;   // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr int kEpilogueThreads = 128;
constexpr int kGroupM = 8;          // pair rows (256 tokens each) per raster group: their X rows stay L2-resident
constexpr int kNumSmsPlanned = 148; // used where the answer must not depend on the device
constexpr int kPairsPlanned = kNumSmsPlanned / 2;
constexpr int kMaxSplits = 16;      // split factor of the shrink along d_in
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct RowGate { float w_in, w_out; int r_in, r_out; };  // g[j] = w_in [j < r_in] + w_out [j < r_out]

struct ApplyParams {
  int T, d_in, d_out, R;   // R = 0: no adapter
  int r_pad;               // R rounded up to 128: each CTA of a pair supplies whole 64-column swizzle atoms
  int n_m_pairs, n_n_tiles;
  int splits, kb_per_split;
  int window;
  __nv_bfloat16* Y; int64_t ldy;
  __nv_bfloat16* Hg;       // [T, R] gated shrink output
  float* partial;          // [splits, T, R]
  int* counters;           // [2 n_m_pairs] splits finished per 128-row tile
  int* flags;              // [2 n_m_pairs] 1 once H' of the 128-row tile is published
  cwl_chunk_table table;
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

// TMA load into THIS CTA's shared memory whose bytes are counted on the pair leader's mbarrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem] across the CTA pair: 256 x N x 16, bf16 in, fp32 out.  Each CTA supplies its
// 128 rows of A and its half of B's columns, and receives its 128 rows of D in its own TMEM.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier at this shared-memory offset arrives in BOTH CTAs once every MMA issued so far has finished
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
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


__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// orders this thread's generic-proxy observations before its later async-proxy (TMA) accesses
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `cta` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t cta) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}

// ------------------------------------------------------------------------------------ work items
enum : int { ITEM_SHRINK = 0, ITEM_PROJECT = 1 };
struct Item { int kind, m_pair, n_tile, split; };

struct SmemPlan {
  static constexpr int kABytes = BM * BK * 2;        // 16 KB: one TMA box of X or H' (this CTA's 128 rows)
  static constexpr int kBBytes = (BN / 2) * BK * 2;  // 16 KB: this CTA's half of the right operand (two 64 x 64 boxes)
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTileBytes = kStages * kStageBytes;
  static constexpr int kBarBytes = (2 * kStages + 4) * 8;
  static constexpr int kMiscBytes = 32;              // TMEM base, abort flag, epilogue broadcast words
  static constexpr int kGateBytes = BM * (int)sizeof(RowGate);
  static constexpr int kTotal = kTileBytes + kBarBytes + kMiscBytes + kGateBytes + 1024;  // + alignment slack
};

// The i-th work item of this CTA pair.  A pair owns 256 rows (CTA rank r the rows 128 r .. 128 r + 127).
// Shrink items come first and are dealt from the LAST pair downwards, so the pairs that receive one
// projection tile fewer carry the shrink work.  Projection tiles are rastered in groups of kGroupM pair
// rows (pair row fastest inside a group) so a group's X rows and the W column slabs stay in L2.
__device__ __forceinline__ bool get_item(int i, const ApplyParams& p, Item& it) {
  const int G = gridDim.x >> 1, b = blockIdx.x >> 1;
  const int n_shrink = (p.R > 0) ? p.n_m_pairs * p.splits : 0;
  const int first_s = G - 1 - b;
  const int my_shrink = first_s < n_shrink ? (n_shrink - 1 - first_s) / G + 1 : 0;
  if (i < my_shrink) {
    const int s = first_s + i * G;
    it.kind = ITEM_SHRINK; it.m_pair = s / p.splits; it.split = s - it.m_pair * p.splits; it.n_tile = 0;
    return true;
  }
  const int tile = b + (i - my_shrink) * G;
  if (tile >= p.n_m_pairs * p.n_n_tiles) return false;
  const int per_group = kGroupM * p.n_n_tiles;
  const int group = tile / per_group, within = tile - group * per_group;
  const int first_m = group * kGroupM;
  const int gsize = min(kGroupM, p.n_m_pairs - first_m);
  it.kind = ITEM_PROJECT; it.split = 0;
  it.m_pair = first_m + within % gsize;
  it.n_tile = within / gsize;
  return true;
}

// Pipeline steps of an item: shrink = its split of the d_in blocks; project = all d_in blocks, then R blocks.
__device__ __forceinline__ void item_blocks(const Item& it, const ApplyParams& p, int& kb0, int& n0, int& n1) {
  const int nkb0 = (p.d_in + BK - 1) / BK;
  if (it.kind == ITEM_SHRINK) {
    kb0 = it.split * p.kb_per_split;
    n0 = min(nkb0, kb0 + p.kb_per_split) - kb0;
    n1 = 0;
  } else {
    kb0 = 0; n0 = nkb0; n1 = (p.R + BK - 1) / BK;
  }
}

// Per-row gate from the chunk table (Sec. III-C rank mask and scale, Sec. III-D cross-fade weight).
__device__ __forceinline__ RowGate row_gate(int t, const ApplyParams& p) {
  RowGate g{0.f, 0.f, 0, 0};
  const cwl_chunk_table& tb = p.table;
  const int C = min(*tb.n_chunks, tb.capacity);
  if (t < p.T && C > 0 && t >= tb.offsets[0] && t < tb.offsets[C]) {
    int lo = 0, hi = C;                            // offsets[lo] <= t < offsets[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (tb.offsets[mid] <= t) lo = mid; else hi = mid;
    }
    const int c = lo, j = t - tb.offsets[c];
    float lam = 1.f;
    if (c > 0 && !(tb.flags[c] & 1) && j < p.window) lam = (float)(j + 1) / (float)(p.window + 1);
    g.r_in = min(max(tb.rank[c], 0), p.R);
    g.w_in = lam * tb.scale[c];
    if (lam < 1.f) {
      g.r_out = min(max(tb.rank[c - 1], 0), p.R);
      g.w_out = (1.f - lam) * tb.scale[c - 1];
    }
  }
  return g;
}
__device__ __forceinline__ float gate_at(const RowGate& g, int j) {
  return (j < g.r_in ? g.w_in : 0.f) + (j < g.r_out ? g.w_out : 0.f);
}

// Bounded acquire-wait on a row tile's "H' published" flag.
__device__ __forceinline__ bool wait_flag(const int* flag, volatile int* abort_flag) {
  if (ld_acquire(flag) != 0) return true;
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (ld_acquire(flag) != 0) return true;
    __nanosleep(64);
    if ((spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
apply_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
             const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_h,
             const __grid_constant__ CUtensorMap tm_b, const ApplyParams p) {
  using Plan = SmemPlan;
  constexpr uint32_t kTmemCols = 2 * BN;            // two accumulators: all 512 columns

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;     // swizzled tiles need 1024-byte alignment
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bars = base + Plan::kTileBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bars + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * kStages + 2 + a); };
  uint8_t* misc = base_ptr + Plan::kTileBytes + Plan::kBarBytes;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  volatile int* epi_go = reinterpret_cast<volatile int*>(misc + 8);     // epilogue: proceed with this item?
  volatile int* epi_last = reinterpret_cast<volatile int*>(misc + 12);  // epilogue: this CTA finalises the row tile
  RowGate* gates = reinterpret_cast<RowGate*>(misc + Plan::kMiscBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair (issues the MMAs)

  if (threadIdx.x == 0) {
    // full: armed by the leader's producer, completed by both CTAs' TMA bytes (only the leader's copy is used)
    // empty / acc_full: one arrival from the leader's tcgen05.commit, multicast to both CTAs
    // acc_empty: the 128 epilogue threads of BOTH CTAs arrive on the leader's copy
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 2 * kEpilogueThreads); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm_x);
    prefetch_tmap(&tm_w);
    if (p.R > 0) { prefetch_tmap(&tm_a); prefetch_tmap(&tm_h); prefetch_tmap(&tm_b); }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();                                   // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t it_cnt = 0;      // running stage counter across items
      bool ok = true;
      Item item;
      for (int i = 0; ok && get_item(i, p, item); ++i) {
        int kb0, n0, n1;
        item_blocks(item, p, kb0, n0, n1);
        const bool shrink = item.kind == ITEM_SHRINK;
        const int m_tile = item.m_pair * 2 + (int)rank;       // this CTA's 128-row tile
        const int half = shrink ? p.r_pad / 2 : BN / 2;       // columns of the right operand this CTA supplies
        const int n_boxes = half / 64;
        const uint32_t tx_pair = 2u * (Plan::kABytes + n_boxes * (BK * 128));
        const CUtensorMap* right0 = shrink ? &tm_a : &tm_w;
        const int col0 = (shrink ? 0 : item.n_tile * BN) + (int)rank * half;
        for (int b = 0; b < n0 + n1; ++b, ++it_cnt) {
          const int s = it_cnt % kStages;
          const uint32_t ph = (it_cnt / kStages) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const bool phase1 = b >= n0;
          if (phase1 && b == n0) {
            // H' of this CTA's row tile must have been published by whoever finished its shrink
            if (!wait_flag(p.flags + m_tile, abort_flag)) { ok = false; break; }
            fence_proxy_async();
          }
          const int k = phase1 ? (b - n0) * BK : (kb0 + b) * BK;
          const CUtensorMap* left = phase1 ? &tm_h : &tm_x;
          const CUtensorMap* right = phase1 ? &tm_b : right0;
          const uint32_t sa = base + s * Plan::kStageBytes, sb = sa + Plan::kABytes;
          const uint32_t leader_full = full_bar(s) & 0xFEFFFFFFu;   // the same barrier in the leader's shared memory
          if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
          tma_load_2d_pair(sa, left, leader_full, k, m_tile * BM);
          for (int j = 0; j < n_boxes; ++j)
            tma_load_2d_pair(sb + j * (BK * 128), right, leader_full, col0 + j * 64, k);
        }
      }
      if (!ok && rank == 0) {
        // drain: give the copies already issued a bounded chance to land before the CTA leaves
        for (uint32_t back = 1; back <= (uint32_t)kStages && back <= it_cnt; ++back) {
          const uint32_t j = it_cnt - back;
          unsigned long long t0 = global_timer();
          while (!mbar_try_wait(full_bar(j % kStages), (j / kStages) & 1u) && global_timer() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc_project = make_idesc(2 * BM, BN);
      const uint32_t idesc_shrink = make_idesc(2 * BM, p.r_pad > 0 ? p.r_pad : 128);
      uint32_t it_cnt = 0, local = 0;
      bool ok = true;
      Item item;
      for (int i = 0; ok && get_item(i, p, item); ++i, ++local) {
        int kb0, n0, n1;
        item_blocks(item, p, kb0, n0, n1);
        const uint32_t idesc = item.kind == ITEM_SHRINK ? idesc_shrink : idesc_project;
        const uint32_t acc = local & 1u, acc_ph = (local >> 1) & 1u;
        if (!mbar_wait(acc_empty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int b = 0; b < n0 + n1; ++b, ++it_cnt) {
          const int s = it_cnt % kStages;
          const uint32_t ph = (it_cnt / kStages) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const bool phase1 = b >= n0;
          const int k = phase1 ? (b - n0) * BK : (kb0 + b) * BK;
          const int k_left = (phase1 ? p.R : p.d_in) - k;          // multiple of 16
          const int k_steps = k_left >= BK ? BK / UMMA_K : k_left / UMMA_K;
          const uint32_t sa = base + s * Plan::kStageBytes, sb = sa + Plan::kABytes;
          for (int kk = 0; kk < k_steps; ++kk) {
            const uint64_t da = make_smem_desc(sa + kk * (UMMA_K * 2), 16, 1024);
            const uint64_t db = make_smem_desc(sb + kk * (UMMA_K * 128), BK * 128, 1024);
            umma_bf16_pair(d_tmem, da, db, idesc, (b | kk) != 0 ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(s));            // frees the stage in both CTAs once these MMAs have read it
        }
        if (ok) umma_commit_pair(acc_full_bar(acc)); // accumulator complete, both CTAs
      }
      if (!ok) {
        // give the MMAs still in flight a bounded time to retire before TMEM is released
        unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 1000000ull) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int lane_group = warp & 3;              // TMEM lanes this warp may read: 32*lane_group ..
    const int row_in_tile = lane_group * 32 + lane;
    const int epi_tid = threadIdx.x - 64;         // 0..127
    uint32_t local = 0;
    Item item;
    for (int i = 0; get_item(i, p, item); ++i, ++local) {
      const uint32_t acc = local & 1u, acc_ph = (local >> 1) & 1u;
      mbar_wait(acc_full_bar(acc), acc_ph, abort_flag);   // a failure is recorded in abort_flag
      // one thread decides for all 128 so that the barriers below are never split
      epilogue_barrier();
      if (epi_tid == 0) *epi_go = (*abort_flag == 0);
      epilogue_barrier();
      if (*epi_go == 0) break;
      tc_fence_after();
      const int m_tile = item.m_pair * 2 + (int)rank;
      const int row = m_tile * BM + row_in_tile;
      const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(lane_group * 32) << 16);
      const uint32_t leader_acc_empty = mapa_shared(acc_empty_bar(acc), 0);

      if (item.kind == ITEM_PROJECT) {
#pragma unroll 1
        for (int cc = 0; cc < BN / 32; ++cc) {
          const int col = item.n_tile * BN + cc * 32;
          if (col >= p.d_out) break;                 // warp-uniform
          uint32_t v[32];
          tmem_ld32(t_row + cc * 32, v);
          tmem_ld_wait();
          if (row < p.T) {
            __nv_bfloat16* out = p.Y + (int64_t)row * p.ldy + col;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (col + g * 8 < p.d_out) {           // d_out is a multiple of 8: a granule is all in or all out
                uint4 q;
                q.x = pack_bf16(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
                q.y = pack_bf16(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
                q.z = pack_bf16(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
                q.w = pack_bf16(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
                *reinterpret_cast<uint4*>(out + g * 8) = q;
              }
            }
          }
        }
        tc_fence_before();
        mbar_arrive_cluster(leader_acc_empty);
        continue;
      }

      // ---- shrink item ----
      const bool direct = p.splits == 1;             // no partials: gate straight from the accumulator
      RowGate g{0.f, 0.f, 0, 0};
      if (direct) g = row_gate(row, p);
#pragma unroll 1
      for (int cc = 0; cc < p.r_pad / 32; ++cc) {
        const int col = cc * 32;
        if (col >= p.R) break;                       // warp-uniform
        uint32_t v[32];
        tmem_ld32(t_row + cc * 32, v);
        tmem_ld_wait();
        if (row < p.T) {
          if (direct) {
            __nv_bfloat16* out = p.Hg + (int64_t)row * p.R + col;
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              if (col + q8 * 8 < p.R) {
                const int j = col + q8 * 8;
                uint4 q;
                q.x = pack_bf16(__uint_as_float(v[q8 * 8 + 0]) * gate_at(g, j + 0), __uint_as_float(v[q8 * 8 + 1]) * gate_at(g, j + 1));
                q.y = pack_bf16(__uint_as_float(v[q8 * 8 + 2]) * gate_at(g, j + 2), __uint_as_float(v[q8 * 8 + 3]) * gate_at(g, j + 3));
                q.z = pack_bf16(__uint_as_float(v[q8 * 8 + 4]) * gate_at(g, j + 4), __uint_as_float(v[q8 * 8 + 5]) * gate_at(g, j + 5));
                q.w = pack_bf16(__uint_as_float(v[q8 * 8 + 6]) * gate_at(g, j + 6), __uint_as_float(v[q8 * 8 + 7]) * gate_at(g, j + 7));
                *reinterpret_cast<uint4*>(out + q8 * 8) = q;
              }
            }
          } else {
            float* out = p.partial + ((int64_t)item.split * p.T + row) * p.R + col;
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              if (col + q4 * 4 < p.R)
                *reinterpret_cast<uint4*>(out + q4 * 4) = make_uint4(v[q4 * 4 + 0], v[q4 * 4 + 1], v[q4 * 4 + 2], v[q4 * 4 + 3]);
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive_cluster(leader_acc_empty);         // the accumulator is free again

      __threadfence();                               // this thread's H' / partial stores, device-wide
      epilogue_barrier();
      if (direct) {
        if (epi_tid == 0) st_release(p.flags + m_tile, 1);
        continue;
      }
      if (epi_tid == 0) *epi_last = (atomicAdd(p.counters + m_tile, 1) == p.splits - 1);
      epilogue_barrier();
      if (*epi_last == 0) continue;
      // this CTA completed its row tile: sum the partials, gate, publish H'
      __threadfence();
      gates[epi_tid] = row_gate(m_tile * BM + epi_tid, p);
      epilogue_barrier();
      const int quads = p.R >> 2;                    // float4 groups per row
      const int64_t split_stride = (int64_t)p.T * p.R;
      for (int idx = epi_tid; idx < BM * quads; idx += kEpilogueThreads) {
        const int r = idx / quads, j0 = (idx - r * quads) << 2;
        const int t = m_tile * BM + r;
        if (t >= p.T) break;
        const RowGate gr = gates[r];
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* src = p.partial + (int64_t)t * p.R + j0;
        for (int s = 0; s < p.splits; ++s) {
          const float4 x = __ldcg(reinterpret_cast<const float4*>(src + s * split_stride));
          sum.x += x.x; sum.y += x.y; sum.z += x.z; sum.w += x.w;
        }
        uint2 o;
        o.x = pack_bf16(sum.x * gate_at(gr, j0), sum.y * gate_at(gr, j0 + 1));
        o.y = pack_bf16(sum.z * gate_at(gr, j0 + 2), sum.w * gate_at(gr, j0 + 3));
        *reinterpret_cast<uint2*>(p.Hg + (int64_t)t * p.R + j0) = o;
      }
      __threadfence();
      epilogue_barrier();
      if (epi_tid == 0) st_release(p.flags + m_tile, 1);
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync();   // neither CTA leaves (or frees TMEM) while the other may still signal it or write its TMEM
  if (threadIdx.x == 0 && *abort_flag) flag_status(p.status_word, CWL_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
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

// CTA pairs that can be resident at once (clusters of 2 need both SMs in one GPC)
int max_pairs() {
  static int n = []() {
    int v = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * kPairsPlanned, 1, 1);
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = SmemPlan::kTotal;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemPlan::kTotal) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&v, apply_kernel, &cfg) != cudaSuccess || v <= 0) {
      cudaGetLastError();
      v = sm_count() / 2;
    }
    if (getenv("CWL_LOG") != nullptr) fprintf(stderr, "[cwl] resident CTA pairs: %d (SMs %d)\n", v, sm_count());
    return v;
  }();
  return n;
}

// split factor of the shrink along d_in: enough items to spread X over the SMs when T is small
int shrink_splits(int T, int d_in) {
  const int n_pairs = ceil_div(T, 2 * BM), nkb = ceil_div(d_in, BK);
  int s = kPairsPlanned / n_pairs;
  if (s > kMaxSplits) s = kMaxSplits;
  if (s > nkb) s = nkb;
  if (s < 1) s = 1;
  const int per = ceil_div(nkb, s);
  return ceil_div(nkb, per);        // no empty split
}

struct ApplyWorkspace { __nv_bfloat16* Hg; float* partial; int* counters; int* flags; size_t sync_bytes; };

size_t carve_apply(ApplyWorkspace& w, char* base, int T, int d_in, int R) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const int splits = shrink_splits(T, d_in), n_m = 2 * ceil_div(T, 2 * BM);
  size_t off = 0;
  w.Hg = reinterpret_cast<__nv_bfloat16*>(base ? base + off : nullptr);
  off = up(off + (size_t)T * R * sizeof(__nv_bfloat16));
  w.partial = reinterpret_cast<float*>(base ? base + off : nullptr);
  if (splits > 1) off = up(off + (size_t)splits * T * R * sizeof(float));
  w.counters = reinterpret_cast<int*>(base ? base + off : nullptr);
  w.flags = w.counters + n_m;
  w.sync_bytes = sizeof(int) * 2 * (size_t)n_m;
  off = up(off + w.sync_bytes);
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
  if (adapter && (table.offsets == nullptr || table.rank == nullptr || table.scale == nullptr ||
                  table.flags == nullptr || table.n_chunks == nullptr || table.capacity < 0))
    return CWL_ERR_INVALID_ARG;
  if (T == 0) return CWL_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);

  ApplyWorkspace ws{nullptr, nullptr, nullptr, nullptr, 0};
  if (adapter) {
    const size_t need = carve_apply(ws, static_cast<char*>(workspace), T, d_in, R);
    if (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
      return CWL_ERR_WORKSPACE;
  }

  CUtensorMap mX, mW, mA, mH, mB;
  if (!make_map(&mX, X, (uint64_t)d_in, (uint64_t)T, (uint64_t)ldx, BK, BM)) return CWL_ERR_CUDA;
  if (!make_map(&mW, W, (uint64_t)d_out, (uint64_t)d_in, (uint64_t)ldw, 64, BK)) return CWL_ERR_CUDA;
  if (adapter) {
    if (!make_map(&mA, A, (uint64_t)R, (uint64_t)d_in, (uint64_t)lda, 64, BK)) return CWL_ERR_CUDA;
    if (!make_map(&mH, ws.Hg, (uint64_t)R, (uint64_t)T, (uint64_t)R, BK, BM)) return CWL_ERR_CUDA;
    if (!make_map(&mB, B, (uint64_t)d_out, (uint64_t)R, (uint64_t)ldb, 64, BK)) return CWL_ERR_CUDA;
  } else {
    mA = mW; mH = mX; mB = mW;   // never dereferenced when R == 0
  }

  ApplyParams p{};
  p.T = T; p.d_in = d_in; p.d_out = d_out; p.R = adapter ? R : 0;
  p.r_pad = adapter ? ceil_div(R, 128) * 128 : 0;
  p.n_m_pairs = ceil_div(T, 2 * BM); p.n_n_tiles = ceil_div(d_out, BN);
  p.splits = adapter ? shrink_splits(T, d_in) : 1;
  p.kb_per_split = ceil_div(ceil_div(d_in, BK), p.splits);
  p.window = window;
  p.Y = static_cast<__nv_bfloat16*>(Y); p.ldy = ldy;
  p.Hg = ws.Hg; p.partial = ws.partial; p.counters = ws.counters; p.flags = ws.flags;
  p.table = table; p.status_word = status_word;

  // the per-row-tile counters and flags are the only words that must start at zero
  if (adapter) CWL_CUDA_TRY(cudaMemsetAsync(ws.counters, 0, ws.sync_bytes, stream));

  static bool configured[64] = {};  // per device; benign race: the attribute call is idempotent
  int dev = 0;
  CWL_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    CWL_CUDA_TRY(cudaFuncSetAttribute(apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemPlan::kTotal));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const int items = p.n_m_pairs * p.n_n_tiles, pairs_max = max_pairs();
  const int pairs = items < pairs_max ? items : pairs_max;
  apply_kernel<<<2 * pairs, kGemmThreads, SmemPlan::kTotal, stream>>>(mX, mW, mA, mH, mB, p);
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
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
