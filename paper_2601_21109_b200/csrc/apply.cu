// cwl_apply: adapted projection (Sec. III-F) with the boundary cross-fade (Sec. III-D).
//
//   y_t = x_t W + ((x_t A) * g_t) B,   g_t[j] = (1-lam_t) s_p [j < r_p] + lam_t s_c [j < r_c]
//
// which, by linearity, equals blending the outgoing and incoming adapter outputs.  ONE persistent,
// warp-specialised kernel does all of it, launched as clusters of two CTAs.  A pair owns 256 rows and
// issues tcgen05.mma with cta_group::2: each CTA stages its 128 rows of the left operand and HALF of
// the right operand per pipeline step.  With 256 x 256 tiles the main loop is bound by the rate at which
// operands reach shared memory (measured: ~89 GB/s per SM with the MMAs taken out, 32 KB per 64-deep K
// block), so output tiles are as wide as tensor memory allows: up to 256 x 512 per pair (one accumulator
// of 512 fp32 columns per CTA, two MMAs per K step that share the left operand).  That needs 25 % fewer
// operand bytes per FLOP and puts the loop on the MMA side of the balance (0.64 us of MMAs against
// 0.54 us of operand delivery per K block); the real kernel runs within 3-10 % of its MMAs alone.
//
// Work items of a pair, in order:
//   SHRINK   P[split] = X[:, split of d_in] A[split, :]  at the full ladder rank R, one item per projection
//            (fp32 partials when d_in is split); the CTA that completes a row tile's last split sums the partials, applies
//            the per-row gate (rank mask, scale and cross-fade weight from the chunk table, expanded per
//            row in shared memory) and publishes H' = bf16(g * X A) with a release flag.  The host-side
//            plan hands shrink items to the pairs with the lightest projection load.
//   PROJECT  Y tile = bf16([X | H'] [W ; B]): the K loop runs over d_in and then over R into the SAME
//            accumulator (the TMA producer acquires the row tile's flag before its first H' load).
//            Column tiles come in two widths (wide ones first, then narrower ones that fill the last
//            wave); items are dealt round-robin.  Up to four projections that read the same rows can share
//            one launch (their tiles and shrink items are dealt together).  When the whole problem is a fraction of one wave
//            (decode-sized T) the K loop of each tile is split over several pairs instead: each writes
//            an fp32 partial, and once all of a tile's partials are in, every contributor reduces its
//            share of the tile's columns and writes Y.
//
// Roles per CTA: warp 0 = TMA producer (cp.async.bulk.tensor, 128-byte swizzle, bytes counted on the
// leader's mbarrier), warp 1 = tcgen05.mma issuer in the leader CTA only (tcgen05.commit multicast
// frees the stage in both CTAs), warps 2..9 = epilogue (tcgen05.ld of the CTA's own 128 accumulator
// rows; two warps per TMEM lane quadrant).  The left operand is K-major (rows of X / H'), the right
// operand is N-major (rows of W, A, B are contiguous in their output dimension), exactly as the
// matrices sit in HBM.
//
// Every wait (mbarrier, flag or counter) is bounded: when it runs out the CTA raises CWL_ERR_TIMEOUT in
// the status word, drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <random>
#include <unordered_map>

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int BM = 128;             // rows per CTA tile = TMEM lanes
constexpr int BK = 64;              // K elements per stage = one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int kMaxTileW = 512;      // widest column tile = all TMEM columns
constexpr int kMmaN = 256;          // widest single MMA across the pair
constexpr int kBoxCols = 64;        // columns of one right-operand TMA box (one swizzle atom)
constexpr int kABytes = BM * BK * 2;          // 16 KB: this CTA's 128 rows of the left operand
constexpr int kBoxBytes = kBoxCols * BK * 2;  // 8 KB
constexpr int kMaxStages = 8;
constexpr int kRingBytes = 192 * 1024;
// A launch whose tiles split their K loop never stages whole output tiles, so its epilogue needs the row gates only:
// the operand ring takes the room (one more 40 KB stage in flight for 336- and 384-wide decode tiles).
constexpr int kRingBytesSplit = 216 * 1024;
constexpr int kOutBytesSplit = 8 * 1024;
constexpr int kOutBufBytes = 4096;  // per epilogue warp: 32 rows x 64 bf16 columns staged for row-contiguous stores
constexpr int kThreads = 320;       // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..9: epilogue
constexpr int kEpiThreads = 256;
constexpr int kEpiWarps = 8;
constexpr int kGroupM = 16;         // pair rows (256 tokens each) per raster group: a wave of tiles shares them (see raster())
constexpr int kPairsPlanned = 74;   // most CTA pairs ever launched (148 SMs); plans never use more
constexpr int kMaxSplits = 16;      // split factor of the shrink along d_in
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct RowGate { float w_in, w_out; int r_in, r_out; };  // g[j] = w_in [j < r_in] + w_out [j < r_out]

// Host-side schedule of one launch.  Everything the device needs to enumerate its items.
struct Plan {
  int pairs;                  // CTA pairs launched
  int n_m_pairs;              // 256-row tiles
  int nkb0, nkb1;             // K blocks over d_in, over R
  int n_proj;                 // projections sharing X and the chunk table (1 for cwl_apply)
  int d_out[CWL_MAX_GROUP];   // their output widths
  int w0, n_wide;             // wide column tiles per pair row, all projections together
  int w1, n_narrow;           // narrow tiles per pair row, all projections together
  int pw[CWL_MAX_GROUP];      // projection j: columns [0, pw[j] * w0) in wide tiles,
  int pn[CWL_MAX_GROUP];      //               then pn[j] tiles of width w1 (the last tile of a projection may be ragged)
  int split_k, kb_per_ksplit; // split of the d_in blocks of every tile (1 = none); only when all items fit one wave
  int shrink_splits, kb_per_split;
  int boxes;                  // right-operand boxes per CTA per stage, at most
  int stages;
  uint16_t sh_count[kPairsPlanned];  // shrink items per pair
  long long makespan;         // model cost of the busiest pair (diagnostic)
};

struct ApplyParams {
  int T, d_in, R;          // R = 0: no adapter
  int RT;                  // n_proj * R: columns of the shrink output, all projections side by side
  int window;
  int window_mode;         // CWL_WINDOW_CAUSAL: the window follows the join; CWL_WINDOW_CENTRED: it lies around it
  __nv_bfloat16* Y[CWL_MAX_GROUP]; int64_t ldy[CWL_MAX_GROUP];
  __nv_bfloat16* Hg;       // [T, RT] gated shrink outputs
  float* partial;          // [shrink_splits, 128-row tiles, RT / 4, 128, 4] fp32 partial shrink sums
  float* sk_partial;       // [tiles * split_k * 2, 128, w0] fp32 partial accumulators of split-K items
  // Sync words are 64 bits: (epoch of the launch << 8) | count.  A word that carries another epoch (left by an earlier
  // launch, or never written) counts as zero, so nothing has to be cleared between launches.
  unsigned long long* counters;     // [2 n_m_pairs][n_proj] shrink splits finished per (128-row tile, projection)
  unsigned long long* flags;        // [2 n_m_pairs][n_proj] 1 once that projection's H' columns of the row tile are published
  unsigned long long* sk_counters;  // [2 tiles] split-K partials stored per (tile, CTA rank)
  unsigned long long epoch;         // this launch's tag, already shifted: low 8 bits zero
  cwl_chunk_table table;
  const cwl_row_gate* row_gates;   // when set: one descriptor per row instead of the chunk table
  unsigned long long wait_limit_ns; // limit of every device-side wait
  const unsigned char* pf_ptr;      // hinted region the NEXT call will stream (its weights), 128-byte aligned; or null
  unsigned long long pf_bytes;      // its size, a multiple of 128
  int withhold_publish;            // test hook: never publish H', so that the waits on it run out
  int32_t* status_word;
  Plan plan;
};

// Tensor maps of one launch: X and H' are shared, the rest is per projection.
struct GroupMaps {
  CUtensorMap x, h;
  CUtensorMap w[CWL_MAX_GROUP], a[CWL_MAX_GROUP], b[CWL_MAX_GROUP];
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// The CTA's wait limit in ns sits 12 bytes after its abort flag in shared memory (set once at kernel start).
__device__ __forceinline__ unsigned long long wait_limit(volatile int* abort_flag) {
  return *reinterpret_cast<volatile unsigned long long*>(abort_flag + 3);
}
#ifdef CWL_TEST_HOOKS
// Test build only (cwl_trace_set): the leader CTA of one chosen pair writes %globaltimer readings of its producer, its
// MMA issuer and its first epilogue thread into a caller-supplied array; the slots are listed in cwl_test_hooks.h.
__device__ long long* g_trace = nullptr;
__device__ int g_trace_pair = -1;
#define CWL_TRACE_DECL const bool tr = g_trace != nullptr && (int)(blockIdx.x >> 1) == g_trace_pair && cluster_ctarank() == 0
#define CWL_TRACE(i) do { if (tr) g_trace[(i)] = (long long)global_timer(); } while (0)
#define CWL_TRACE_N(base, i) do { if (tr && (i) < 290u) g_trace[(base) + (i)] = (long long)global_timer(); } while (0)
#else
#define CWL_TRACE_DECL do {} while (0)
#define CWL_TRACE(i) do {} while (0)
#define CWL_TRACE_N(base, i) do {} while (0)
#endif

// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > wait_limit(abort_flag)) { *abort_flag = 1; return false; }
    }
  }
}

// TMA load into THIS CTA's shared memory whose bytes are counted on the pair leader's mbarrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y) : "memory");
}
// The same with an L2 eviction policy for the lines it brings in.
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y,
                                                      uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y), "l"(policy) : "memory");
}
// L2 eviction policies: rows of X are read again by every column tile of their raster group (keep them), rows of Y are
// written once and not read by this launch (let them go first).  W gets no hint when several row tiles share its column slabs:
// the pairs that share a slab read it within a short time of one another, and marking it for early eviction was measured to
// double its DRAM reads.  With one row tile (decode) every box is read once and is marked to leave first.
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void st_global_v4_hint(void* ptr, uint4 v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;"
               ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(policy) : "memory");
}
// contiguous global -> shared copy (16-byte aligned, a multiple of 16 bytes) counted on an mbarrier of this CTA
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// asks L2 for a contiguous run of global memory (16-byte aligned, a multiple of 16 bytes); no destination, no completion
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
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

__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// count carried by a sync word for the launch tagged `epoch` (another tag: zero)
__device__ __forceinline__ int sync_count(unsigned long long word, unsigned long long epoch) {
  return ((word ^ epoch) >> 8) == 0 ? (int)(word & 0xffu) : 0;
}
// One more arrival on a sync word; returns the count before it.  Lock-free: an attempt fails only because another
// arrival succeeded, and a word sees at most a few dozen arrivals per launch.
__device__ __forceinline__ int sync_arrive(unsigned long long* word, unsigned long long epoch) {
  unsigned long long old = *reinterpret_cast<volatile unsigned long long*>(word);
  for (;;) {
    const unsigned long long cur = ((old ^ epoch) >> 8) == 0 ? old : epoch;
    const unsigned long long seen = atomicCAS(word, old, cur + 1);
    if (seen == old) return (int)(cur & 0xffu);
    old = seen;
  }
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
__host__ __device__ __forceinline__ int boxes_for(int cols_per_cta) { return (cols_per_cta + kBoxCols - 1) / kBoxCols; }

enum : int { ITEM_SHRINK = 0, ITEM_PROJECT = 1 };
struct Item {
  int kind, m_pair;
  int proj;             // project: which projection of the group
  int n0, wt;           // first column and width (multiple of 16) of the tile; shrink: 0, R
  int split;            // shrink: which split of d_in.  project: which K split
  int tile;             // project: index of the output tile (for split-K bookkeeping)
  int kb0, n_blk0;      // d_in blocks [kb0, kb0 + n_blk0)
  int n_blk1;           // then this many R blocks (project items that own the end of the K loop)
  int wa, wb;           // widths of the two MMAs (wb may be 0): columns [n0, n0+wa) and [n0+wa, n0+wt)
};

// Rastered tile index -> (pair row, column tile): groups of kGroupM pair rows, pair row fastest inside a
// group.  The 74 tiles in flight then cover 16 pair rows x 4-5 column tiles, close to the smallest set of X rows and
// W slabs 74 tiles can touch (about 50 MB at d_in = 4096), and the next 74 need the same X rows again.
__device__ __forceinline__ void raster(int tile, int n_m_pairs, int n_cols, int& m_pair, int& c) {
  const int per_group = kGroupM * n_cols;
  const int group = tile / per_group, within = tile - group * per_group;
  const int first_m = group * kGroupM;
  const int gsize = min(kGroupM, n_m_pairs - first_m);
  m_pair = first_m + within % gsize;
  c = within / gsize;
}

__device__ __forceinline__ void set_widths(Item& it) {
  it.wa = min(it.wt, kMmaN);
  it.wb = it.wt - it.wa;
}

// The i-th work item of CTA pair `b` (shrink items first).
__device__ __forceinline__ bool get_item(int i, int b, int sh_begin, const ApplyParams& p, Item& it) {
  const Plan& pl = p.plan;
  const int my_shrink = pl.sh_count[b];
  if (i < my_shrink) {
    const int s = sh_begin + i, per_row = pl.n_proj * pl.shrink_splits;   // one item per (row tile, projection, split)
    it.kind = ITEM_SHRINK; it.m_pair = s / per_row;
    const int rem = s - it.m_pair * per_row;
    it.proj = rem / pl.shrink_splits; it.split = rem - it.proj * pl.shrink_splits;
    it.n0 = 0; it.wt = p.R; it.tile = 0;
    it.kb0 = it.split * pl.kb_per_split;
    it.n_blk0 = min(pl.nkb0, it.kb0 + pl.kb_per_split) - it.kb0;
    it.n_blk1 = 0;
    set_widths(it);
    return true;
  }
  const int idx = b + (i - my_shrink) * pl.pairs;
  const int n_wide_tiles = pl.n_m_pairs * pl.n_wide, n_narrow_tiles = pl.n_m_pairs * pl.n_narrow;
  const int n_tiles = n_wide_tiles + n_narrow_tiles;
  if (idx >= n_tiles * pl.split_k) return false;
  const int tile = idx / pl.split_k, ks = idx - tile * pl.split_k;
  int c, w, j = 0;
  if (tile < n_wide_tiles) {
    raster(tile, pl.n_m_pairs, pl.n_wide, it.m_pair, c);
    while (c >= pl.pw[j]) { c -= pl.pw[j]; ++j; }
    it.n0 = c * pl.w0; w = pl.w0;
  } else {
    raster(tile - n_wide_tiles, pl.n_m_pairs, pl.n_narrow, it.m_pair, c);
    while (c >= pl.pn[j]) { c -= pl.pn[j]; ++j; }
    it.n0 = pl.pw[j] * pl.w0 + c * pl.w1; w = pl.w1;
  }
  it.kind = ITEM_PROJECT; it.tile = tile; it.split = ks; it.proj = j;
  it.wt = min(w, pl.d_out[j] - it.n0);         // d_out and the widths are multiples of 16
  it.kb0 = ks * pl.kb_per_ksplit;
  it.n_blk0 = min(pl.nkb0, it.kb0 + pl.kb_per_ksplit) - it.kb0;
  it.n_blk1 = (ks == pl.split_k - 1) ? pl.nkb1 : 0;
  set_widths(it);
  return true;
}

// Per-row gate from the chunk table (Sec. III-C rank mask and scale, Sec. III-D cross-fade weight).
__device__ __forceinline__ RowGate row_gate(int t, const ApplyParams& p) {
  RowGate g{0.f, 0.f, 0, 0};
  if (p.row_gates != nullptr) {
    if (t < p.T) {
      const cwl_row_gate d = p.row_gates[t];
      g.r_in = min(max(d.rank_in, 0), p.R);
      g.w_in = d.lambda * d.scale_in;
      if (d.lambda < 1.f) {
        g.r_out = min(max(d.rank_out, 0), p.R);
        g.w_out = (1.f - d.lambda) * d.scale_out;
      }
    }
    return g;
  }
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
    int c_in = c, c_out = c;                       // configurations carrying lam and 1 - lam
    if (p.window_mode == CWL_WINDOW_CENTRED) {
      // the window lies around the join: floor(w/2) rows before it, ceil(w/2) rows after it; where a short chunk's
      // two windows meet, the rows belong to the join that opened the chunk
      const int before = p.window >> 1, after = p.window - before;
      const int len = tb.offsets[c + 1] - tb.offsets[c];
      if (c > 0 && !(tb.flags[c] & 1) && j < after) {
        lam = (float)(before + j + 1) / (float)(p.window + 1);
        c_out = c - 1;
      } else if (c + 1 < C && !(tb.flags[c + 1] & 1) && len - j <= before) {
        lam = (float)(before - (len - j) + 1) / (float)(p.window + 1);
        c_in = c + 1;
      }
    } else if (c > 0 && !(tb.flags[c] & 1) && j < p.window) {
      lam = (float)(j + 1) / (float)(p.window + 1);
      c_out = c - 1;
    }
    g.r_in = min(max(tb.rank[c_in], 0), p.R);
    g.w_in = lam * tb.scale[c_in];
    if (lam < 1.f) {
      g.r_out = min(max(tb.rank[c_out], 0), p.R);
      g.w_out = (1.f - lam) * tb.scale[c_out];
    }
  }
  return g;
}
__device__ __forceinline__ float gate_at(const RowGate& g, int j) {
  return (j < g.r_in ? g.w_in : 0.f) + (j < g.r_out ? g.w_out : 0.f);
}

// Bounded acquire-wait until *word >= target.
__device__ __forceinline__ bool wait_word(const unsigned long long* word, unsigned long long epoch, int target,
                                          volatile int* abort_flag) {
  if (sync_count(ld_acquire(word), epoch) >= target) return true;
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (sync_count(ld_acquire(word), epoch) >= target) return true;
    __nanosleep(64);
    if ((spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > wait_limit(abort_flag)) { *abort_flag = 1; return false; }
    }
  }
}

struct SmemLayout {
  static constexpr int kOutBytes = kEpiWarps * kOutBufBytes;   // also holds the row gates of a shrink finaliser
  static constexpr int kBarBytes = (2 * kMaxStages + 3) * 8;
  static constexpr int kMiscBytes = 32;              // TMEM base, abort flag, epilogue broadcast words
  static constexpr int kTotal = kRingBytes + kOutBytes + kBarBytes + kMiscBytes + 1024;  // + alignment slack
};
static_assert(BM * sizeof(RowGate) <= SmemLayout::kOutBytes && BM * sizeof(RowGate) <= kOutBytesSplit, "row gates must fit the staging area");
static_assert(kRingBytesSplit + kOutBytesSplit == kRingBytes + SmemLayout::kOutBytes, "both instantiations use the same amount of shared memory");
static_assert(SmemLayout::kTotal <= 227 * 1024, "shared memory budget");

// Two instantiations: kSplitK = false for plans whose tiles keep their whole K loop (the epilogue stores whole
// tiles), kSplitK = true for plans that split every tile's K loop over several pairs (the epilogue hands partial
// accumulators over).  A launch runs exactly one of the two epilogues, so neither carries the other's code.
template <bool kSplitK>
__device__ __forceinline__ void apply_body(const GroupMaps& tm, const ApplyParams& p, const int pair) {
  using L = SmemLayout;
  constexpr uint32_t kTmemCols = kMaxTileW;

  // Programmatic dependent launch: the next launch of this stream may place its CTAs as soon as this grid's CTAs
  // leave their SMs; it waits below, after its set-up, until this grid has completed and its writes are visible.
  // (Both instructions do nothing in a launch made without the attribute.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;     // swizzled tiles need 1024-byte alignment
  uint8_t* base_ptr = smem_raw + (base - raw);
  constexpr int kRing = kSplitK ? kRingBytesSplit : kRingBytes;
  constexpr int kOut = kSplitK ? kOutBytesSplit : L::kOutBytes;
  const uint32_t out_bufs = base + kRing;           // per-warp staging buffers of the epilogue
  const uint32_t bars = out_bufs + kOut;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
  const uint32_t acc_full_bar = bars + 8u * (2 * kMaxStages);
  const uint32_t acc_empty_bar = bars + 8u * (2 * kMaxStages + 1);
  const uint32_t fix_bar = bars + 8u * (2 * kMaxStages + 2);   // split-K: the others' partial sums have landed
  uint8_t* misc = base_ptr + kRing + kOut + L::kBarBytes;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  volatile int* epi_go = reinterpret_cast<volatile int*>(misc + 8);     // epilogue: proceed with this item?
  volatile int* epi_last = reinterpret_cast<volatile int*>(misc + 12);  // epilogue: this CTA finalises the row tile
  RowGate* gates = reinterpret_cast<RowGate*>(base_ptr + kRing);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair (issues the MMAs)
  const Plan& pl = p.plan;
  const int n_stages = pl.stages;
  const uint32_t stage_bytes = kABytes + pl.boxes * kBoxBytes;

  if (threadIdx.x == 0) {
    // full: armed by the leader's producer, completed by both CTAs' TMA bytes (only the leader's copy is used)
    // empty / acc_full: one arrival from the leader's tcgen05.commit, multicast to both CTAs
    // acc_empty: one arrival per epilogue warp of BOTH CTAs, on the leader's copy
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(acc_full_bar, 1);
    mbar_init(acc_empty_bar, 2 * kEpiWarps);
    mbar_init(fix_bar, 1);
    *abort_flag = 0;
    *reinterpret_cast<volatile unsigned long long*>(abort_flag + 3) = p.wait_limit_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tm.x);
    for (int j = 0; j < p.plan.n_proj; ++j) {
      prefetch_tmap(&tm.w[j]);
      if (p.R > 0) { prefetch_tmap(&tm.a[j]); prefetch_tmap(&tm.b[j]); }
    }
    if (p.R > 0) prefetch_tmap(&tm.h);
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
  int sh_begin = 0;                                 // first shrink item of this pair
  for (int g = 0; g < pair; ++g) sh_begin += pl.sh_count[g];
  {
    // Decoding a work item reads only kernel parameters.  Doing it once before waiting for the launch ahead in the
    // stream takes the constant-cache misses of the plan out of the time between that launch's end and the first load.
    Item warm;
    const bool any = get_item(0, pair, sh_begin, p, warm);
    asm volatile("" ::"r"(warm.wt + warm.kb0 + warm.n_blk0 + warm.n0 + (any ? 1 : 0)));
  }
  CWL_TRACE_DECL;
  if (threadIdx.x == 32) CWL_TRACE(0);
  asm volatile("griddepcontrol.wait;" ::: "memory");   // nothing before this line reads or writes global memory (but a trace)
  if (threadIdx.x == 32) CWL_TRACE(1);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    // The whole warp walks the ring; per K block lane 0 arms the barrier and loads the left operand, lanes 1..n
    // load one right-operand box each, so the copies of a step go out with one instruction instead of a chain.
    {
      if (lane == 0) CWL_TRACE(19);
      uint32_t it_cnt = 0;      // running stage counter across items
      uint32_t s = 0, ph = 0;   // ring slot and phase parity of it_cnt, kept incrementally (no division per step)
      const uint32_t leader_full0 = mapa_shared(full_bar(0), 0);   // full_bar(0) in the leader's shared memory
      bool ok = true;
      const uint64_t keep_x = policy_evict_last();
      // With a single row tile (decode-sized T) every box of W or A is read by exactly one pair, once: let it leave L2 first,
      // so that the rows of X, the partial sums and H' stay.  With more row tiles the pairs of a raster group share the box.
      const bool stream_w = pl.n_m_pairs == 1;
      const uint64_t drop_w = policy_evict_first();
      Item item;
      for (int i = 0; ok && get_item(i, pair, sh_begin, p, item); ++i) {
        const bool shrink = item.kind == ITEM_SHRINK;
        const int m_tile = item.m_pair * 2 + (int)rank;       // this CTA's 128-row tile
        // columns of the right operand this CTA supplies: its half of each MMA's columns (a shrink item runs one
        // MMA of N = R against its projection's A, a projection tile one or two MMAs)
        const int ca = item.wa >> 1, cb = item.wb >> 1;
        const int boxes_a = boxes_for(ca), boxes_b = boxes_for(cb);
        const int col_a = item.n0 + (int)rank * ca;
        const int col_b = item.n0 + item.wa + (int)rank * cb;
        const int n_boxes = boxes_a + boxes_b;
        const uint32_t tx_pair = 2u * (kABytes + n_boxes * kBoxBytes);
        // this lane's box (lanes 1..n_boxes): source matrix in the d_in blocks and in the R blocks, column, slot
        const int bi = lane - 1;
        const bool has_box = bi >= 0 && bi < n_boxes;
        const CUtensorMap* map0 = shrink ? &tm.a[item.proj] : &tm.w[item.proj];
        const CUtensorMap* map1 = &tm.b[item.proj];
        int box_x = 0;
        if (has_box) box_x = bi < boxes_a ? col_a + bi * kBoxCols : col_b + (bi - boxes_a) * kBoxCols;
        const int n_blk = item.n_blk0 + item.n_blk1;
        if (lane == 0 && it_cnt == 0) CWL_TRACE(20);
        for (int b = 0; b < n_blk; ++b, ++it_cnt) {
          bool step_ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag);
          if (lane == 0 && it_cnt == 0) CWL_TRACE(21);
          const bool phase1 = b >= item.n_blk0;
          if (phase1 && b == item.n_blk0) {
            // H' of this CTA's row tile must have been published by whoever finished its shrink
            if (lane == 0) CWL_TRACE(15);
            if (lane == 0 && step_ok) step_ok = wait_word(p.flags + m_tile * pl.n_proj + item.proj, p.epoch, 1, abort_flag);
            if (lane == 0) CWL_TRACE(16);
            fence_proxy_async();
          }
          if (!__all_sync(0xffffffffu, step_ok)) { ok = false; break; }
          const int k = phase1 ? (b - item.n_blk0) * BK : (item.kb0 + b) * BK;
          const uint32_t sa = base + s * stage_bytes, sb = sa + kABytes;
          const uint32_t leader_full = leader_full0 + 8u * s;      // this stage's barrier in the leader's shared memory
          if (lane == 0) {
            CWL_TRACE_N(100, it_cnt);
            if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
            if (phase1) tma_load_2d_pair(sa, &tm.h, leader_full, item.proj * p.R + k, m_tile * BM);
            else tma_load_2d_pair_hint(sa, &tm.x, leader_full, k, m_tile * BM, keep_x);
          } else if (has_box) {
            if (stream_w && !phase1) tma_load_2d_pair_hint(sb + bi * kBoxBytes, map0, leader_full, box_x, k, drop_w);
            else tma_load_2d_pair(sb + bi * kBoxBytes, phase1 ? map1 : map0, leader_full, box_x, k);
          }
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
        }
      }
      if (ok && p.pf_bytes != 0) {
        // All of this CTA's loads are issued.  From here to the end of the launch (the last K blocks, the hand-over of
        // partial sums, the output stores) and through the start of the next launch HBM would sit idle: ask L2 for this
        // CTA's slice of the region the caller says the next call streams.  Read-only, no completion to wait for.
        constexpr unsigned long long kPiece = 8192;
        const unsigned long long n_cta = gridDim.x;
        unsigned long long slice = (p.pf_bytes + n_cta - 1) / n_cta;
        slice = (slice + 127ull) & ~127ull;
        const unsigned long long lo = (unsigned long long)blockIdx.x * slice;
        const unsigned long long hi = lo + slice < p.pf_bytes ? lo + slice : p.pf_bytes;
        for (unsigned long long off = lo + (unsigned long long)lane * kPiece; off < hi; off += 32ull * kPiece) {
          const unsigned long long n = hi - off < kPiece ? hi - off : kPiece;
          bulk_prefetch_l2(p.pf_ptr + off, (uint32_t)n);
        }
      }
      if (!ok && rank == 0 && lane == 0) {
        // drain: give the copies already issued a bounded chance to land before the CTA leaves
        for (uint32_t back = 1; back <= (uint32_t)n_stages && back <= it_cnt; ++back) {
          const uint32_t j = it_cnt - back;
          unsigned long long t0 = global_timer();
          while (!mbar_try_wait(full_bar(j % n_stages), (j / n_stages) & 1u) && global_timer() - t0 < wait_limit(abort_flag)) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    // One thread issues every MMA of the pair, so the instructions it executes per K block are on the critical path
    // of narrow (decode-sized) tiles, whose tensor-core time per block is short: device timestamps showed 0.47 us from
    // "operands landed" to "commit issued" for eight MMAs, more than the MMAs themselves take.  The loop therefore
    // keeps running shared-memory descriptors (one 64-bit add per ring slot and per K step instead of rebuilding
    // them), takes the common case of a full 64-deep block through an unrolled path, and works the K extent of the
    // last block of each phase out once per item.
    if (lane == 0 && rank == 0) {
      uint32_t local = 0;
      uint32_t s = 0, ph = 0;   // ring slot and phase parity, kept incrementally
      bool ok = true;
      Item item;
#ifdef CWL_TEST_HOOKS
      uint32_t blocks_done = 0;   // K blocks issued so far, over all items (trace slots)
#endif
      // descriptors of ring slot 0; a slot is stage_bytes further on (the address field counts 16-byte units and the
      // whole ring lies below 256 KB, so adding to the 64-bit descriptor never carries out of the field)
      const uint64_t desc_a0 = make_smem_desc(base, 16, 1024);
      const uint64_t desc_b0 = make_smem_desc(base + kABytes, kBoxBytes, 1024);
      const uint64_t desc_slot = (uint64_t)(stage_bytes >> 4);
      constexpr uint64_t kStepA = (UMMA_K * 2) >> 4;        // one K step further in a K-major tile
      constexpr uint64_t kStepB = (UMMA_K * 128) >> 4;      // ... in an N-major box
      uint64_t da = desc_a0, db = desc_b0;
      for (int i = 0; ok && get_item(i, pair, sh_begin, p, item); ++i, ++local) {
        const uint32_t idesc_a = make_idesc(2 * BM, item.wa);
        const uint32_t idesc_b = make_idesc(2 * BM, item.wb > 0 ? item.wb : 16);
        const uint64_t second = (uint64_t)((uint32_t)boxes_for(item.wa >> 1) * kBoxBytes >> 4);   // second MMA's boxes
        const bool two = item.wb > 0;
        if (!mbar_wait(acc_empty_bar, (local & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const int n_blk = item.n_blk0 + item.n_blk1;
        // K steps of the last block of the d_in phase (if this item holds the end of d_in) and of the R phase
        const int tail0 = (item.kb0 + item.n_blk0 == pl.nkb0 && (p.d_in & (BK - 1)) != 0) ? (p.d_in & (BK - 1)) / UMMA_K : BK / UMMA_K;
        const int tail1 = (p.R & (BK - 1)) != 0 ? (p.R & (BK - 1)) / UMMA_K : BK / UMMA_K;
        for (int b = 0; b < n_blk; ++b) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          CWL_TRACE_N(400, blocks_done);
          tc_fence_after();
          int k_steps = BK / UMMA_K;
          if (b == item.n_blk0 - 1) k_steps = tail0;
          else if (b == n_blk - 1 && item.n_blk1 > 0) k_steps = tail1;
          const uint32_t acc0 = b != 0 ? 1u : 0u;
          if (k_steps == BK / UMMA_K) {
            if (two) {
#pragma unroll
              for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                umma_bf16_pair(tmem_base, da + kk * kStepA, db + kk * kStepB, idesc_a, kk ? 1u : acc0);
                umma_bf16_pair(tmem_base + kMmaN, da + kk * kStepA, db + second + kk * kStepB, idesc_b, kk ? 1u : acc0);
              }
            } else {
#pragma unroll
              for (int kk = 0; kk < BK / UMMA_K; ++kk)
                umma_bf16_pair(tmem_base, da + kk * kStepA, db + kk * kStepB, idesc_a, kk ? 1u : acc0);
            }
          } else {
            for (int kk = 0; kk < k_steps; ++kk) {
              umma_bf16_pair(tmem_base, da + kk * kStepA, db + kk * kStepB, idesc_a, kk ? 1u : acc0);
              if (two) umma_bf16_pair(tmem_base + kMmaN, da + kk * kStepA, db + second + kk * kStepB, idesc_b, kk ? 1u : acc0);
            }
          }
          umma_commit_pair(empty_bar(s));            // frees the stage in both CTAs once these MMAs have read it
#ifdef CWL_TEST_HOOKS
          CWL_TRACE_N(700, blocks_done);
          ++blocks_done;
#endif
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; da = desc_a0; db = desc_b0; }
          else { da += desc_slot; db += desc_slot; }
        }
        if (ok) umma_commit_pair(acc_full_bar);      // accumulator complete, both CTAs
        CWL_TRACE(2);
      }
      if (!ok) {
        // give the MMAs still in flight a bounded time to retire before TMEM is released
        unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 1000000ull) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int quad = warp & 3;                    // TMEM lanes this warp may read: 32*quad .. 32*quad+31
    const int chalf = (warp - 2) >> 2;            // the two warps of a quadrant take alternate 32-column chunks
    const int row_in_tile = quad * 32 + lane;
    const int epi_tid = threadIdx.x - 64;         // 0..255
    const uint32_t leader_acc_empty = mapa_shared(acc_empty_bar, 0);
    uint32_t local = 0;
    Item item;
    for (int i = 0; get_item(i, pair, sh_begin, p, item); ++i, ++local) {
      if (item.kind == ITEM_SHRINK && epi_tid < BM) {
        // the row gates of this item's row tile, looked up while the main loop runs (a chain of dependent loads)
        gates[epi_tid] = row_gate((item.m_pair * 2 + (int)rank) * BM + epi_tid, p);
      }
      mbar_wait(acc_full_bar, local & 1u, abort_flag);    // a failure is recorded in abort_flag
      if (threadIdx.x == 64) CWL_TRACE(5);
      // one thread decides for all 256 so that the barriers below are never split
      epilogue_barrier();
      if (epi_tid == 0) *epi_go = (*abort_flag == 0);
      epilogue_barrier();
      if (*epi_go == 0) break;
      tc_fence_after();
      const int m_tile = item.m_pair * 2 + (int)rank;
      const int row = m_tile * BM + row_in_tile;
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
      const int n_chunks = (item.wt + 31) >> 5;

      if (!kSplitK && item.kind == ITEM_PROJECT) {
        // ---- whole tile: accumulator -> bf16 -> swizzled staging buffer (a lane holds a row) -> read back so that
        // a warp instruction stores four whole 128-byte row segments ----
        const uint32_t obuf = out_bufs + (uint32_t)(warp - 2) * kOutBufBytes;
        const int n64 = item.wt >> 6;                // whole 64-column chunks
        const int row0 = m_tile * BM + quad * 32;
#pragma unroll 1
        for (int c64 = chalf; c64 < n64; c64 += 2) {
          __syncwarp();                              // every lane has read the previous chunk back
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld32(t_row + c64 * 64 + h * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 q;
              q.x = pack_bf16(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
              q.y = pack_bf16(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
              q.z = pack_bf16(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
              q.w = pack_bf16(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
              const int piece = h * 4 + g;           // 16-byte piece of this lane's 128-byte row
              st_shared_v4(obuf + lane * 128 + ((piece ^ (lane & 7)) << 4), q);
            }
          }
          __syncwarp();
          __nv_bfloat16* out = p.Y[item.proj] + item.n0 + c64 * 64 + (lane & 7) * 8;
          const int64_t ldy = p.ldy[item.proj];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int r = (lane >> 3) + 4 * k;       // lanes 8j..8j+7 take the eight pieces of row r
            const uint4 q = ld_shared_v4(obuf + r * 128 + (((lane & 7) ^ (r & 7)) << 4));
            if (row0 + r < p.T) st_global_v4_hint(out + (int64_t)(row0 + r) * ldy, q, policy_evict_first());
          }
        }
        const int rem = item.wt & 63;                // a last chunk of 16, 32 or 48 columns: plain 16-byte stores
        if (rem != 0 && (n64 & 1) == chalf) {
#pragma unroll 1
          for (int h = 0; h * 32 < rem; ++h) {
            uint32_t v[32];
            tmem_ld32(t_row + n64 * 64 + h * 32, v);
            tmem_ld_wait();
            if (row < p.T) {
              __nv_bfloat16* out = p.Y[item.proj] + (int64_t)row * p.ldy[item.proj] + item.n0 + n64 * 64 + h * 32;
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                if (h * 32 + g * 8 < rem) {
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
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
        continue;
      }

      if (kSplitK && item.kind == ITEM_PROJECT) {
        // ---- split-K item: every contributor owns a share of the tile's columns.  It stores the OTHER columns of
        // its fp32 accumulator (layout [column group of 4][128 rows][4]: a warp's store and the owner's loads are
        // contiguous), waits until all partials of the tile are in, and adds the others' partials of its own
        // share to what is still in its tensor memory.  This is the pair's last item, so the accumulator is not
        // handed back before the end, and the operand ring is free: the bf16 result is staged there row by row
        // and written to Y with contiguous 16-byte stores.
        const int share = (((item.wt + pl.split_k - 1) / pl.split_k) + 7) & ~7;
        const int c_lo = min(item.wt, item.split * share), c_hi = min(item.wt, c_lo + share);
        const int pitch = share * 2 + 16;            // bytes per staged row
        float* tile_base = p.sk_partial + ((int64_t)(item.tile * pl.split_k) * 2 + rank) * (BM * pl.w0);
        const int64_t split_stride = (int64_t)2 * BM * pl.w0;
        float* mine = tile_base + item.split * split_stride;
#pragma unroll 1
        for (int cc = chalf; cc < n_chunks; cc += 2) {
          if (cc * 32 >= c_lo && cc * 32 + 32 <= c_hi) continue;   // wholly mine (warp-uniform)
          uint32_t v[32];
          tmem_ld32(t_row + cc * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const int col = cc * 32 + q4 * 4;
            if (col < item.wt && (col < c_lo || col >= c_hi))
              *reinterpret_cast<uint4*>(mine + ((cc * 8 + q4) * BM + row_in_tile) * 4) =
                  make_uint4(v[q4 * 4 + 0], v[q4 * 4 + 1], v[q4 * 4 + 2], v[q4 * 4 + 3]);
          }
        }
        epilogue_barrier();                          // every thread's partial stores precede thread 0's release below
        if (threadIdx.x == 64) CWL_TRACE(6);
        unsigned long long* counter = p.sk_counters + item.tile * 2 + rank;
        // The others' partial sums of this CTA's share are one contiguous run per contributor: where they fit the
        // (now idle) operand ring beside the staged rows, bulk copies bring them in at once instead of a chain of
        // dependent loads per thread.
        const uint32_t seg_bytes = (uint32_t)(c_hi - c_lo) * (BM * 4);          // one contributor's run
        const uint32_t land = ((uint32_t)(BM * pitch) + 1023u) & ~1023u;        // offset of the landing zone in the ring
        const bool landed = c_hi > c_lo && land + (uint32_t)(pl.split_k - 1) * seg_bytes <= (uint32_t)kRing;
        if (epi_tid == 0) {
          __threadfence();                           // device-wide release of the CTA's partial (cumulative over the barrier)
          sync_arrive(counter, p.epoch);
          bool in = wait_word(counter, p.epoch, pl.split_k, abort_flag);
          CWL_TRACE(7);
          if (in && landed) {
            fence_proxy_async();                     // the partials were written with ordinary stores
            mbar_expect_tx(fix_bar, (uint32_t)(pl.split_k - 1) * seg_bytes);
            int slot = 0;
            for (int s = 0; s < pl.split_k; ++s) {
              if (s == item.split) continue;
              bulk_load(base + land + slot * seg_bytes, tile_base + s * split_stride + (int64_t)(c_lo >> 2) * (BM * 4), seg_bytes, fix_bar);
              ++slot;
            }
            in = mbar_wait(fix_bar, 0, abort_flag);  // bounded; a failure is recorded in abort_flag
          }
          *epi_go = in ? 1 : 0;
          CWL_TRACE(8);
        }
        epilogue_barrier();
        if (*epi_go == 0) break;
        if (landed) mbar_wait(fix_bar, 0, abort_flag);   // completed already: every thread observes the copies itself
        else __threadfence();
#pragma unroll 1
        for (int cc = (c_lo >> 5) + ((((c_lo >> 5) & 1) != chalf) ? 1 : 0); cc * 32 < c_hi; cc += 2) {
          uint32_t v[32];
          tmem_ld32(t_row + cc * 32, v);
          tmem_ld_wait();
          float acc[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[j] = __uint_as_float(v[j]);
          if (landed) {
            // landing zone: [contributor][column group of 4 from c_lo][128 rows][4]
            const uint32_t l0 = base + land + (uint32_t)(((cc * 8 - (c_lo >> 2)) * BM + row_in_tile) * 16);
#pragma unroll 1
            for (int slot = 0; slot < pl.split_k - 1; ++slot) {
#pragma unroll
              for (int q4 = 0; q4 < 8; ++q4) {
                const int col = cc * 32 + q4 * 4;
                if (col >= c_lo && col < c_hi) {
                  const uint4 x = ld_shared_v4(l0 + slot * seg_bytes + q4 * (BM * 16));
                  acc[q4 * 4 + 0] += __uint_as_float(x.x); acc[q4 * 4 + 1] += __uint_as_float(x.y);
                  acc[q4 * 4 + 2] += __uint_as_float(x.z); acc[q4 * 4 + 3] += __uint_as_float(x.w);
                }
              }
            }
          } else {
            const float* src0 = tile_base + ((int64_t)(cc * 8) * BM + row_in_tile) * 4;
#pragma unroll 2
            for (int s = 0; s < pl.split_k; ++s) {
              if (s == item.split) continue;
              const float* src = src0 + s * split_stride;
#pragma unroll
              for (int q4 = 0; q4 < 8; ++q4) {
                const int col = cc * 32 + q4 * 4;
                if (col >= c_lo && col < c_hi) {
                  const float4 x = __ldcg(reinterpret_cast<const float4*>(src + q4 * BM * 4));
                  acc[q4 * 4 + 0] += x.x; acc[q4 * 4 + 1] += x.y; acc[q4 * 4 + 2] += x.z; acc[q4 * 4 + 3] += x.w;
                }
              }
            }
          }
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const int col = cc * 32 + q4 * 4;
            if (col >= c_lo && col < c_hi) {
              uint2 o;
              o.x = pack_bf16(acc[q4 * 4 + 0], acc[q4 * 4 + 1]);
              o.y = pack_bf16(acc[q4 * 4 + 2], acc[q4 * 4 + 3]);
              *reinterpret_cast<uint2*>(base_ptr + row_in_tile * pitch + (col - c_lo) * 2) = o;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
        epilogue_barrier();
        if (threadIdx.x == 64) CWL_TRACE(9);
        const int pieces = (c_hi - c_lo) >> 3;       // 16-byte pieces per row
        for (int idx = epi_tid; idx < BM * pieces; idx += kEpiThreads) {
          const int r = idx / pieces, pc = idx - r * pieces;
          const int t = m_tile * BM + r;
          if (t >= p.T) break;
          const uint4 q = *reinterpret_cast<const uint4*>(base_ptr + r * pitch + pc * 16);
          *reinterpret_cast<uint4*>(p.Y[item.proj] + (int64_t)t * p.ldy[item.proj] + item.n0 + c_lo + pc * 8) = q;
        }
        continue;
      }

      // ---- shrink item ----
      const bool direct = pl.shrink_splits == 1;     // no partials: gate straight from the accumulator
      const RowGate g = gates[row_in_tile];          // written before the barriers above
      const int sync_idx = m_tile * pl.n_proj + item.proj;   // counter and flag of this (row tile, projection)
      const int hcol = item.proj * p.R;              // this projection's columns of H'
#pragma unroll 1
      for (int cc = chalf; cc < n_chunks; cc += 2) {
        const int col = cc * 32;
        uint32_t v[32];
        tmem_ld32(t_row + cc * 32, v);
        tmem_ld_wait();
        if (!direct) {
          // partial layout [split][128-row tile][column group of 4][128 rows][4]: contiguous per warp store
          float* out = p.partial + (((int64_t)(item.split * 2 * pl.n_m_pairs + m_tile) * (p.RT >> 2) + (hcol >> 2) + cc * 8) * BM + row_in_tile) * 4;
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            if (col + q4 * 4 < p.R)
              *reinterpret_cast<uint4*>(out + q4 * BM * 4) = make_uint4(v[q4 * 4 + 0], v[q4 * 4 + 1], v[q4 * 4 + 2], v[q4 * 4 + 3]);
          }
        } else if (row < p.T) {
          {
            __nv_bfloat16* out = p.Hg + (int64_t)row * p.RT + hcol + col;
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              if (col + q8 * 8 < p.R) {
                const int j = col + q8 * 8;              // rank index (R is a multiple of 8)
                uint4 q;
                q.x = pack_bf16(__uint_as_float(v[q8 * 8 + 0]) * gate_at(g, j + 0), __uint_as_float(v[q8 * 8 + 1]) * gate_at(g, j + 1));
                q.y = pack_bf16(__uint_as_float(v[q8 * 8 + 2]) * gate_at(g, j + 2), __uint_as_float(v[q8 * 8 + 3]) * gate_at(g, j + 3));
                q.z = pack_bf16(__uint_as_float(v[q8 * 8 + 4]) * gate_at(g, j + 4), __uint_as_float(v[q8 * 8 + 5]) * gate_at(g, j + 5));
                q.w = pack_bf16(__uint_as_float(v[q8 * 8 + 6]) * gate_at(g, j + 6), __uint_as_float(v[q8 * 8 + 7]) * gate_at(g, j + 7));
                *reinterpret_cast<uint4*>(out + q8 * 8) = q;
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_acc_empty);   // the accumulator is free again

      __threadfence();                               // this thread's H' / partial stores, device-wide
      epilogue_barrier();
      if (direct) {
        if (epi_tid == 0 && !p.withhold_publish) st_release(p.flags + sync_idx, p.epoch | 1ull);
        continue;
      }
      if (threadIdx.x == 64) CWL_TRACE(11);
      if (epi_tid == 0) *epi_last = (sync_arrive(p.counters + sync_idx, p.epoch) == pl.shrink_splits - 1);
      epilogue_barrier();
      if (threadIdx.x == 64) CWL_TRACE(12);
      if (*epi_last == 0) continue;
      // this CTA completed its projection's share of the row tile: sum the partials, gate, publish H'
      __threadfence();
      if (threadIdx.x == 64) CWL_TRACE(17);
      const int quads = p.R >> 2;                    // float4 groups per row of this projection
      const int64_t split_stride = (int64_t)2 * pl.n_m_pairs * p.RT * BM;
      // Every thread owns the groups idx = epi_tid + k * 256.  It takes them eight at a time and, split by split, loads
      // the eight partial sums before it adds any of them: the loads of a batch are independent, so their latencies
      // overlap (a loop that finished one group before it loaded the next one took one memory round trip per group).
      constexpr int kBatch = 8;
      for (int idx0 = epi_tid; idx0 < BM * quads; idx0 += kEpiThreads * kBatch) {
        float4 sum[kBatch];
        const float* src[kBatch];
#pragma unroll
        for (int g = 0; g < kBatch; ++g) {
          const int idx = idx0 + g * kEpiThreads;
          const int r = idx & (BM - 1), cg = idx >> 7;
          const bool live = idx < BM * quads && m_tile * BM + r < p.T;
          sum[g] = make_float4(0.f, 0.f, 0.f, 0.f);
          src[g] = live ? p.partial + (((int64_t)m_tile * (p.RT >> 2) + (hcol >> 2) + cg) * BM + r) * 4 : nullptr;
        }
#pragma unroll 2
        for (int s = 0; s < pl.shrink_splits; ++s) {
          float4 x[kBatch];
#pragma unroll
          for (int g = 0; g < kBatch; ++g)
            x[g] = src[g] != nullptr ? __ldcg(reinterpret_cast<const float4*>(src[g] + s * split_stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int g = 0; g < kBatch; ++g) { sum[g].x += x[g].x; sum[g].y += x[g].y; sum[g].z += x[g].z; sum[g].w += x[g].w; }
        }
        if (threadIdx.x == 64) CWL_TRACE(18);
#pragma unroll
        for (int g = 0; g < kBatch; ++g) {
          if (src[g] == nullptr) continue;
          const int idx = idx0 + g * kEpiThreads;
          const int r = idx & (BM - 1), cg = idx >> 7, j0 = cg << 2;   // rank index
          const RowGate gr = gates[r];
          uint2 o;
          o.x = pack_bf16(sum[g].x * gate_at(gr, j0), sum[g].y * gate_at(gr, j0 + 1));
          o.y = pack_bf16(sum[g].z * gate_at(gr, j0 + 2), sum[g].w * gate_at(gr, j0 + 3));
          *reinterpret_cast<uint2*>(p.Hg + (int64_t)(m_tile * BM + r) * p.RT + hcol + j0) = o;
        }
      }
      if (threadIdx.x == 64) CWL_TRACE(13);
      __threadfence();
      epilogue_barrier();
      if (threadIdx.x == 64) CWL_TRACE(14);
      if (epi_tid == 0 && !p.withhold_publish) st_release(p.flags + sync_idx, p.epoch | 1ull);
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (threadIdx.x == 64) CWL_TRACE(3);
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 64) CWL_TRACE(4);
  cluster_sync();   // neither CTA leaves (or frees TMEM) while the other may still signal it or write its TMEM
  if (threadIdx.x == 0 && *abort_flag) flag_status(p.status_word, CWL_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <bool kSplitK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
apply_kernel(const __grid_constant__ GroupMaps tm, const __grid_constant__ ApplyParams p) {
  apply_body<kSplitK>(tm, p, (int)(blockIdx.x >> 1));
}

// Several independent projections in ONE launch (cwl_apply_batch): every projection has its own run of CTA pairs and
// its own plan, operands, workspace and sync words, exactly as if it had been launched alone on that many pairs; a pair
// looks up which projection it belongs to and does that projection's work.  The projections share nothing but the
// launch, so their set-up and their drains overlap one another's main loops, and consecutive batch launches chain like
// any other launch of the library.
struct BatchArgs {
  int n;
  int first_pair[CWL_MAX_BATCH + 1];   // projection j owns pairs [first_pair[j], first_pair[j + 1])
  int split[CWL_MAX_BATCH];            // its plan splits the K loop (which epilogue it runs)
  GroupMaps maps[CWL_MAX_BATCH];
  ApplyParams params[CWL_MAX_BATCH];
};

static_assert(sizeof(BatchArgs) <= 16 * 1024, "kernel parameters of the batch launch");

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
apply_batch_kernel(const __grid_constant__ BatchArgs a) {
  const int gp = (int)(blockIdx.x >> 1);
  int j = 0;
  while (j + 1 < a.n && gp >= a.first_pair[j + 1]) ++j;
  if (a.split[j]) apply_body<true>(a.maps[j], a.params[j], gp - a.first_pair[j]);
  else apply_body<false>(a.maps[j], a.params[j], gp - a.first_pair[j]);
}

// ------------------------------------------------------------------------------- host: the plan
// Cost model, in KB of operands a CTA stages per K block: (16 KB of rows + 8 KB per right-operand box), plus a
// per-tile epilogue term.  (Measured with the loads or the MMAs taken out of the loop, a 512-wide tile is bound by
// its MMAs, 0.64 us per K block against 0.54 us for its 48 KB of operands; a model that credits narrower tiles
// with their shorter MMAs picked 464-wide tiles for 4096 columns on 74 pairs and measured 10 % slower.)
int tile_boxes(int w) {
  const int wa = w < kMmaN ? w : kMmaN, wb = w - wa;
  return boxes_for(wa / 2) + boxes_for(wb / 2);
}
long long tile_cost(int w, int kblocks) { return (long long)kblocks * (16 + 8 * tile_boxes(w)) + w / 4; }

// items idx in [first, first + count) dealt as idx % pairs: how many land on pair g
int dealt(int first, int count, int pairs, int g) {
  auto upto = [&](int n) { return n > g ? (n - 1 - g) / pairs + 1 : 0; };
  return upto(first + count) - upto(first);
}

// split factor of the shrink along d_in: enough items to spread X over the SMs when T is small
int shrink_splits_for(int T, int d_in) {
  const int n_pairs = ceil_div(T, 2 * BM), nkb = ceil_div(d_in, BK);
  int s = kPairsPlanned / n_pairs;
  if (s > kMaxSplits) s = kMaxSplits;
  if (s > nkb) s = nkb;
  if (s < 1) s = 1;
  const int per = ceil_div(nkb, s);
  return ceil_div(nkb, per);        // no empty split
}

// Chooses tile widths, the K split and who does the shrink work for `pairs` resident CTA pairs.
// Depends on the shape and on `pairs` only.  allow_split_k = false keeps every tile whole; scratch_limit > 0
// keeps the shrink's split small enough for H' and the partial sums to fit that many bytes (one split always may).
Plan search_plan(int T, int d_in, int n_proj, const int* d_out, int R, int pairs, bool allow_split_k,
                 size_t scratch_limit) {
  Plan pl;
  memset(&pl, 0, sizeof(pl));
  if (pairs > kPairsPlanned) pairs = kPairsPlanned;
  if (pairs < 1) pairs = 1;
  pl.n_proj = n_proj;
  int max_dout = 0, max_floor = 0;
  for (int j = 0; j < n_proj; ++j) {
    pl.d_out[j] = d_out[j];
    if (d_out[j] > max_dout) max_dout = d_out[j];
    if (d_out[j] / kMaxTileW > max_floor) max_floor = d_out[j] / kMaxTileW;
  }
  pl.n_m_pairs = ceil_div(T, 2 * BM);
  pl.nkb0 = ceil_div(d_in, BK);
  pl.nkb1 = R > 0 ? ceil_div(R, BK) : 0;
  const int kbt = pl.nkb0 + pl.nkb1;
  pl.shrink_splits = R > 0 ? shrink_splits_for(T, d_in) : 1;
  pl.kb_per_split = ceil_div(pl.nkb0, pl.shrink_splits);
  pl.split_k = 1; pl.kb_per_ksplit = pl.nkb0;

  // ---- column tiling.  Candidates: every projection in tiles of one width (512, 496, ... 128; last one ragged), or
  // in tiles of 512 with `drop` fewer of them each and the remaining columns in tiles of w1; or (decode-sized problems: at most half a wave of
  // tiles, one width) every tile's K loop split over several pairs.  The busiest pair's cost decides.
  long long best = -1;
  const int narrow_widths[3] = {256, 384, 128};
  // drop = -1 - u, u = 0..24: one width 512 - 16 u for every tile (each projection's last tile ragged); widths
  // below 512 are candidates for the split-K form only (measured: they help decode, not prefill)
  for (int drop = -25; drop <= max_floor; ++drop) {
    for (int wi = 0; wi < 3; ++wi) {
      int w0 = drop < 0 ? kMaxTileW - 16 * (-1 - drop) : kMaxTileW, w1 = narrow_widths[wi];
      int pw[CWL_MAX_GROUP], pn[CWL_MAX_GROUP], n_wide = 0, n_narrow = 0;
      for (int j = 0; j < n_proj; ++j) {
        if (drop < 0) { pw[j] = ceil_div(d_out[j], w0); pn[j] = 0; }
        else {
          pw[j] = d_out[j] / kMaxTileW - drop;
          if (pw[j] < 0) pw[j] = 0;
          pn[j] = ceil_div(d_out[j] - pw[j] * kMaxTileW, w1);
        }
        n_wide += pw[j]; n_narrow += pn[j];
      }
      if (n_wide == 0) {                                                // one width only: call it the wide one
        w0 = w1; n_wide = n_narrow; n_narrow = 0;
        for (int j = 0; j < n_proj; ++j) { pw[j] = pn[j]; pn[j] = 0; }
      }
      if (w0 > max_dout) w0 = max_dout;                                 // then every projection is a single tile
      const int NW = pl.n_m_pairs * n_wide, NN = pl.n_m_pairs * n_narrow;
      const int used = NW + NN < pairs ? NW + NN : pairs;
      long long worst = 0;
      for (int g = 0; g < used; ++g) {
        const long long load = dealt(0, NW, used, g) * tile_cost(w0, kbt) + dealt(NW, NN, used, g) * tile_cost(w1, kbt);
        if (load > worst) worst = load;
      }
      int split_k = 1, kb_per_ksplit = pl.nkb0;
      if (allow_split_k && n_narrow == 0 && 2 * NW <= pairs) {
        const int spare = pairs >= 16 ? pairs / 9 : 0;   // pairs left free for shrink items (also without an adapter,
                                                         // so that the plan and its workspace do not depend on R)
        int s = (pairs - spare) / NW;
        const int min_kb = 8;                                           // K blocks per item, at least
        if (s > pl.nkb0 / min_kb) s = pl.nkb0 / min_kb;
        if (s > 16) s = 16;
        if (s >= 2) {
          const int per = ceil_div(pl.nkb0, s);
          s = ceil_div(pl.nkb0, per);
          // every contributor stores and later reads (s-1)/s of a 128 x w0 fp32 accumulator through L2; measured
          // (~11 us for w0 = 512, s = 3 against 0.8 us per 48 KB K block) that is worth 2 w0 (s-1)/s staged KB
          const long long c = tile_cost(w0, per + pl.nkb1) + (long long)2 * w0 * (s - 1) / s;
          if (s >= 2 && c < worst) { worst = c; split_k = s; kb_per_ksplit = per; }
        }
      }
      if (drop < -1 && split_k == 1) break;
      if (best < 0 || worst < best) {
        best = worst;
        pl.w0 = w0; pl.n_wide = n_wide; pl.w1 = w1; pl.n_narrow = n_narrow;
        for (int j = 0; j < n_proj; ++j) { pl.pw[j] = pw[j]; pl.pn[j] = pn[j]; }
        pl.split_k = split_k; pl.kb_per_ksplit = kb_per_ksplit;
      }
      if (drop < 0) break;                        // no narrow tiles: their width is irrelevant
    }
  }
  const int n_tiles = pl.n_m_pairs * (pl.n_wide + pl.n_narrow);
  const int n_items = n_tiles * pl.split_k;
  pl.pairs = n_items < pairs ? n_items : pairs;
  if (R > 0 && pl.pairs < pairs) {
    // pairs beyond the projection items exist only to carry shrink items
    const int n_shrink = pl.n_m_pairs * n_proj * pl.shrink_splits;
    pl.pairs = n_items + n_shrink < pairs ? n_items + n_shrink : pairs;
  }

  pl.boxes = tile_boxes(pl.w0);
  if (pl.n_narrow > 0 && tile_boxes(pl.w1) > pl.boxes) pl.boxes = tile_boxes(pl.w1);
  if (R > 0 && boxes_for(R / 2) > pl.boxes) pl.boxes = boxes_for(R / 2);
  pl.stages = (pl.split_k > 1 ? kRingBytesSplit : kRingBytes) / (kABytes + pl.boxes * kBoxBytes);
  if (pl.stages > kMaxStages) pl.stages = kMaxStages;

  // ---- shrink: how finely d_in is split and who does the items.  Items go, one at a time, to the pair with
  // the lightest load so far.  An item costs its K blocks (16 KB of rows + the boxes of A) plus a fixed
  // start-up and hand-over term worth a few K blocks; H' must be there when the first tiles reach the end of
  // their d_in loop, so shrink work that keeps a pair busy beyond that point counts as a stall for everybody.
  long long base_load[kPairsPlanned], load[kPairsPlanned];
  const int NW = pl.n_m_pairs * pl.n_wide * pl.split_k, NN = pl.n_m_pairs * pl.n_narrow;
  const long long cost_w0 = tile_cost(pl.w0, pl.split_k > 1 ? pl.kb_per_ksplit + pl.nkb1 : kbt);
  for (int g = 0; g < pl.pairs; ++g)
    base_load[g] = dealt(0, NW, pl.pairs, g) * cost_w0 + dealt(NW, NN, pl.pairs, g) * tile_cost(pl.w1, kbt);
  long long best_total = -1;
  if (R > 0) {
    const long long first_tile = (long long)(pl.split_k > 1 ? pl.kb_per_ksplit : pl.nkb0) * (16 + 8 * tile_boxes(pl.w0));
    for (int want = 1; want <= kMaxSplits; want *= 2) {
      if (want > pl.nkb0) break;
      const int per = ceil_div(pl.nkb0, want), splits = ceil_div(pl.nkb0, per);
      const size_t RT = (size_t)n_proj * R;
      const size_t scratch = (size_t)T * RT * 2 + (size_t)splits * pl.n_m_pairs * 2 * BM * RT * 4 + 4096 + 32 * (size_t)pl.n_m_pairs * n_proj;
      if (scratch_limit > 0 && splits > 1 && scratch > scratch_limit) continue;
      // measured: a shrink K block costs about 1.3x its staged bytes (narrow MMAs), an item ~4 us of fixed cost
      const long long cs = (long long)per * (16 + 8 * boxes_for(R / 2)) * 13 / 10 + 250;
      const long long due = first_tile * 4 / 5;
      const int n_shrink = pl.n_m_pairs * n_proj * splits;   // one item per (row-tile pair, projection, split)
      uint16_t count[kPairsPlanned];
      long long shrink_time[kPairsPlanned];
      for (int g = 0; g < pl.pairs; ++g) { load[g] = base_load[g]; count[g] = 0; shrink_time[g] = 0; }
      for (int i = 0; i < n_shrink; ++i) {
        // the lightest pair whose shrink work still ends before H' is due; failing that, the one that ends first
        int at = -1;
        for (int g = pl.pairs - 1; g >= 0; --g)
          if (shrink_time[g] + cs <= due && (at < 0 || load[g] < load[at])) at = g;
        if (at < 0) {
          at = pl.pairs - 1;
          for (int g = pl.pairs - 1; g >= 0; --g)
            if (shrink_time[g] < shrink_time[at] || (shrink_time[g] == shrink_time[at] && load[g] < load[at])) at = g;
        }
        load[at] += cs; shrink_time[at] += cs; count[at]++;
      }
      long long worst = 0, latest = 0;
      for (int g = 0; g < pl.pairs; ++g) {
        if (load[g] > worst) worst = load[g];
        if (shrink_time[g] > latest) latest = shrink_time[g];
      }
      const long long total = worst + (latest > due ? 2 * (latest - due) : 0);
      if (best_total < 0 || total < best_total) {
        best_total = total;
        pl.shrink_splits = splits; pl.kb_per_split = per;
        for (int g = 0; g < kPairsPlanned; ++g) pl.sh_count[g] = g < pl.pairs ? count[g] : 0;
      }
    }
    pl.makespan = best_total;
    return pl;
  }
  for (int g = 0; g < pl.pairs; ++g) load[g] = base_load[g];
  pl.makespan = 0;
  for (int g = 0; g < pl.pairs; ++g)
    if (load[g] > pl.makespan) pl.makespan = load[g];
  return pl;
}

// The search costs tens of microseconds of host time, as much as a small launch: plans are remembered per shape.
Plan make_plan(int T, int d_in, int n_proj, const int* d_out, int R, int pairs, bool allow_split_k,
               size_t scratch_limit = 0) {
  struct Key { int v[6 + CWL_MAX_GROUP]; unsigned long long limit; };
  struct Entry { Key key; Plan plan; };
  static std::mutex mu;
  static Entry entries[64];
  static int n_entries = 0, next_slot = 0;
  Key key;
  memset(&key, 0, sizeof(key));
  key.v[0] = T; key.v[1] = d_in; key.v[2] = n_proj; key.v[3] = R; key.v[4] = pairs; key.v[5] = allow_split_k ? 1 : 0;
  for (int j = 0; j < n_proj && j < CWL_MAX_GROUP; ++j) key.v[6 + j] = d_out[j];
  key.limit = scratch_limit;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_entries; ++i)
      if (memcmp(&entries[i].key, &key, sizeof(Key)) == 0) return entries[i].plan;
  }
  const Plan pl = search_plan(T, d_in, n_proj, d_out, R, pairs, allow_split_k, scratch_limit);
  std::lock_guard<std::mutex> lock(mu);
  entries[next_slot].key = key; entries[next_slot].plan = pl;
  next_slot = (next_slot + 1) % 64;
  if (n_entries < 64) ++n_entries;
  return pl;
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

// CTA pairs that can be resident at once (clusters of 2 need both SMs in one GPC); 74 when no device answers
int max_pairs() {
  static int n = []() {
    int v = 0, dev = 0, sms = 2 * kPairsPlanned;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * kPairsPlanned, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = SmemLayout::kTotal;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int v2 = 0;
    if (cudaFuncSetAttribute(apply_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemLayout::kTotal) != cudaSuccess ||
        cudaFuncSetAttribute(apply_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemLayout::kTotal) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&v, apply_kernel<false>, &cfg) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&v2, apply_kernel<true>, &cfg) != cudaSuccess || (v = v < v2 ? v : v2) <= 0) {
      cudaGetLastError();
      v = sms > 0 ? sms / 2 : kPairsPlanned;
    }
    if (v > kPairsPlanned) v = kPairsPlanned;
    if (getenv("CWL_LOG") != nullptr) fprintf(stderr, "[cwl] resident CTA pairs: %d (SMs %d)\n", v, sms);
    return v;
  }();
  return n;
}

// Share of the GPU the calling host thread's apply calls plan for (cwl_set_pair_budget); 0 = all resident pairs.
thread_local int t_pair_budget = 0;
int pairs_now() {
  const int all = max_pairs();
  return t_pair_budget > 0 && t_pair_budget < all ? t_pair_budget : all;
}

// Launch epochs: 56 bits, starting from a per-process random value so that stale words of another process do not
// match either; a word of arbitrary memory matches a given launch with probability 2^-56.
unsigned long long next_epoch() {
  static std::atomic<unsigned long long> counter{[]() {
    std::random_device rd;
    return ((unsigned long long)rd() << 32) ^ (unsigned long long)rd() ^
           (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count();
  }()};
  unsigned long long e;
  do { e = counter.fetch_add(1, std::memory_order_relaxed) & ((1ull << 56) - 1); } while (e == 0);
  return e << 8;
}

// One-shot hint of the calling host thread (cwl_prefetch_next): consumed by its next apply launch.
struct NextPrefetch { const unsigned char* ptr; unsigned long long bytes; };
thread_local NextPrefetch t_next_prefetch = {nullptr, 0};

#ifdef CWL_TEST_HOOKS
// process-wide test hook state (cwl_debug_set); only the test build of the library has it
std::atomic<unsigned long long> g_wait_limit_ns{kWaitLimitNs};
std::atomic<int> g_withhold_publish{0};
#endif

struct ApplyWorkspace { __nv_bfloat16* Hg; float* partial; float* sk_partial; unsigned long long* sync; size_t sync_bytes; };

// Carves the workspace for a plan.
size_t carve_apply(ApplyWorkspace& w, char* base, const Plan& pl, int T, int R) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t RT = (size_t)pl.n_proj * R;
  size_t off = 0;
  w.Hg = reinterpret_cast<__nv_bfloat16*>(base ? base + off : nullptr);
  if (R > 0) off = up(off + (size_t)T * RT * sizeof(__nv_bfloat16));
  w.partial = reinterpret_cast<float*>(base ? base + off : nullptr);
  if (R > 0 && pl.shrink_splits > 1) off = up(off + (size_t)pl.shrink_splits * pl.n_m_pairs * 2 * BM * RT * sizeof(float));
  w.sk_partial = reinterpret_cast<float*>(base ? base + off : nullptr);
  const bool split = pl.split_k > 1;
  const size_t n_tiles = (size_t)pl.n_m_pairs * pl.n_wide;              // split plans have one tile width
  if (split) off = up(off + n_tiles * pl.split_k * 2 * BM * pl.w0 * sizeof(float));
  w.sync = reinterpret_cast<unsigned long long*>(base ? base + off : nullptr);
  // shrink counters [2 n_m][n_proj], H' flags [2 n_m][n_proj], split-K counters [2 tiles]
  w.sync_bytes = sizeof(unsigned long long) * ((size_t)4 * pl.n_m_pairs * pl.n_proj + (split ? 2 * n_tiles : 0));
  off = up(off + w.sync_bytes);
  return off < 256 ? 256 : off;
}

// Argument checks shared by every entry point.  `adapter` comes back true when every projection has both factors.
cwl_status check_group(const void* X, int64_t ldx, const cwl_projection* proj, int n_proj, int T, int d_in, int R,
                       const cwl_chunk_table& table, const cwl_row_gate* row_gates, int window, bool& adapter) {
  if (proj == nullptr || n_proj < 1 || n_proj > CWL_MAX_GROUP) return CWL_ERR_INVALID_ARG;
  if (T < 0 || d_in < 1 || R < 0 || window < 0) return CWL_ERR_INVALID_ARG;
  if (T > 0 && X == nullptr) return CWL_ERR_INVALID_ARG;
  int with = 0;
  for (int j = 0; j < n_proj; ++j) {
    if (proj[j].d_out < 1 || proj[j].W == nullptr || (T > 0 && proj[j].Y == nullptr)) return CWL_ERR_INVALID_ARG;
    if (proj[j].A != nullptr && proj[j].B != nullptr && R > 0) ++with;
  }
  if (with != 0 && with != n_proj) return CWL_ERR_INVALID_ARG;   // adapters on all projections of a group or on none
  adapter = with == n_proj;
  if (d_in % 16 != 0) return CWL_ERR_UNSUPPORTED;
  if (adapter && (R % 16 != 0 || R > CWL_MAX_RANK)) return CWL_ERR_UNSUPPORTED;
  if (ldx < d_in || ldx % 8 != 0 || !aligned16(X)) return CWL_ERR_SHAPE;
  for (int j = 0; j < n_proj; ++j) {
    const cwl_projection& q = proj[j];
    if (q.d_out % 16 != 0) return CWL_ERR_UNSUPPORTED;
    if (q.ldw < q.d_out || q.ldy < q.d_out || (adapter && (q.lda < R || q.ldb < q.d_out))) return CWL_ERR_SHAPE;
    if (q.ldw % 8 != 0 || q.ldy % 8 != 0 || (adapter && (q.lda % 8 != 0 || q.ldb % 8 != 0))) return CWL_ERR_SHAPE;
    if (!aligned16(q.W) || !aligned16(q.Y) || (adapter && (!aligned16(q.A) || !aligned16(q.B)))) return CWL_ERR_SHAPE;
  }
  if (adapter && row_gates == nullptr &&
      (table.offsets == nullptr || table.rank == nullptr || table.scale == nullptr ||
       table.flags == nullptr || table.n_chunks == nullptr || table.capacity < 0))
    return CWL_ERR_INVALID_ARG;
  return CWL_OK;
}

// Plans, carves the workspace, builds the tensor maps and launches one fused kernel for a group of projections.
// Everything one launch (or one projection of a batch launch) needs: plan, carved workspace, tensor maps, parameters.
struct Prepared {
  GroupMaps maps;
  ApplyParams p;
  ApplyWorkspace ws;
  bool uses_sync;          // has sync words (adapter or split K)
};

// Checks the arguments, plans for `pairs` CTA pairs, carves the workspace and builds tensor maps and kernel parameters.
// *launch comes back false when there is nothing to do (T == 0).
cwl_status prepare_group(const void* X, int64_t ldx, const cwl_projection* proj, int n_proj, int32_t T, int32_t d_in,
                         int32_t R, cwl_chunk_table table, int32_t window, void* workspace, size_t workspace_bytes,
                         int32_t* status_word, int pairs, bool allow_split_k, size_t scratch_limit,
                         const cwl_row_gate* row_gates, int32_t window_mode, Prepared& out, bool* launch) {
  *launch = false;
  bool adapter = false;
  const cwl_status chk = check_group(X, ldx, proj, n_proj, T, d_in, R, table, row_gates, window, adapter);
  if (chk != CWL_OK) return chk;
  if (T == 0) return CWL_OK;
  const int Reff = adapter ? R : 0;
  int d_out[CWL_MAX_GROUP];
  for (int j = 0; j < n_proj; ++j) d_out[j] = proj[j].d_out;

  ApplyWorkspace ws{nullptr, nullptr, nullptr, nullptr, 0};
  Plan pl = make_plan(T, d_in, n_proj, d_out, Reff, pairs, allow_split_k, scratch_limit);
  const size_t need = carve_apply(ws, static_cast<char*>(workspace), pl, T, Reff);
  const bool have_ws = workspace != nullptr && workspace_bytes >= need && (reinterpret_cast<uintptr_t>(workspace) & 255u) == 0;
  if (!have_ws && !adapter && pl.split_k > 1) {
    // the plain projection needs scratch only when its K loop is split; without a workspace it runs unsplit
    pl = make_plan(T, d_in, n_proj, d_out, Reff, pairs, false, scratch_limit);
  } else if (!have_ws && (adapter || pl.split_k > 1)) {
    return CWL_ERR_WORKSPACE;
  }

  GroupMaps& maps = out.maps;
  memset(&maps, 0, sizeof(maps));
  if (!make_map(&maps.x, X, (uint64_t)d_in, (uint64_t)T, (uint64_t)ldx, BK, BM)) return CWL_ERR_CUDA;
  maps.h = maps.x;                                  // never dereferenced when R == 0
  if (adapter && !make_map(&maps.h, ws.Hg, (uint64_t)n_proj * R, (uint64_t)T, (uint64_t)n_proj * R, BK, BM)) return CWL_ERR_CUDA;
  for (int j = 0; j < n_proj; ++j) {
    const cwl_projection& q = proj[j];
    if (!make_map(&maps.w[j], q.W, (uint64_t)q.d_out, (uint64_t)d_in, (uint64_t)q.ldw, kBoxCols, BK)) return CWL_ERR_CUDA;
    maps.a[j] = maps.w[j]; maps.b[j] = maps.w[j];   // never dereferenced when R == 0
    if (adapter) {
      if (!make_map(&maps.a[j], q.A, (uint64_t)R, (uint64_t)d_in, (uint64_t)q.lda, kBoxCols, BK)) return CWL_ERR_CUDA;
      if (!make_map(&maps.b[j], q.B, (uint64_t)q.d_out, (uint64_t)R, (uint64_t)q.ldb, kBoxCols, BK)) return CWL_ERR_CUDA;
    }
  }

  ApplyParams& p = out.p;
  p = ApplyParams{};
  p.T = T; p.d_in = d_in; p.R = Reff; p.RT = n_proj * Reff;
  p.window = window; p.window_mode = window_mode;
  for (int j = 0; j < n_proj; ++j) { p.Y[j] = static_cast<__nv_bfloat16*>(proj[j].Y); p.ldy[j] = proj[j].ldy; }
  p.Hg = ws.Hg; p.partial = ws.partial; p.sk_partial = ws.sk_partial;
  p.counters = ws.sync; p.flags = ws.sync + 2 * pl.n_m_pairs * n_proj; p.sk_counters = ws.sync + 4 * pl.n_m_pairs * n_proj;
  p.table = table; p.row_gates = row_gates; p.status_word = status_word;
#ifdef CWL_TEST_HOOKS
  p.wait_limit_ns = g_wait_limit_ns.load(); p.withhold_publish = g_withhold_publish.load();
#else
  p.wait_limit_ns = kWaitLimitNs; p.withhold_publish = 0;
#endif
  p.plan = pl;
  // Every launch tags its sync words with a fresh epoch, so words left by earlier launches (or never written) read as
  // zero and the workspace needs no clearing: a memset between two kernels costs ~5 us of idle GPU.  Only a launch
  // that is being captured into a CUDA graph is replayed with the same epoch; it records a clearing node instead.
  p.epoch = next_epoch();
  out.ws = ws;
  out.uses_sync = adapter || pl.split_k > 1;
  *launch = true;
  return CWL_OK;
}

cwl_status configure_kernels() {
  static bool configured[64] = {};  // per device; benign race: the attribute calls are idempotent
  int dev = 0;
  CWL_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    CWL_CUDA_TRY(cudaFuncSetAttribute(apply_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemLayout::kTotal));
    CWL_CUDA_TRY(cudaFuncSetAttribute(apply_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemLayout::kTotal));
    CWL_CUDA_TRY(cudaFuncSetAttribute(apply_batch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemLayout::kTotal));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  return CWL_OK;
}

// The kernel-to-kernel gap of a stream (~5 us for this cluster launch) is hidden by letting the launch overlap
// the tail of whatever kernel precedes it in the stream; the kernel itself waits for that kernel to complete
// before it touches global memory.  Captured launches keep the plain stream order.
void launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute& attr, int pairs, cudaStream_t stream, bool capturing) {
  cfg = cudaLaunchConfig_t{};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = SmemLayout::kTotal;
  cfg.stream = stream;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = capturing ? 0 : 1;
}

// Plans, carves the workspace, builds the tensor maps and launches one fused kernel for a group of projections.
cwl_status apply_group_impl(const void* X, int64_t ldx, const cwl_projection* proj, int n_proj, int32_t T,
                            int32_t d_in, int32_t R, cwl_chunk_table table, int32_t window, void* workspace,
                            size_t workspace_bytes, int32_t* status_word, void* stream_, bool allow_split_k,
                            size_t scratch_limit, const cwl_row_gate* row_gates = nullptr,
                            int32_t window_mode = CWL_WINDOW_CAUSAL) {
  // the calling thread's one-shot prefetch hint belongs to this call, whatever becomes of it
  const NextPrefetch hint = t_next_prefetch;
  t_next_prefetch = {nullptr, 0};
  Prepared pr;
  bool launch = false;
  const cwl_status st = prepare_group(X, ldx, proj, n_proj, T, d_in, R, table, window, workspace, workspace_bytes,
                                      status_word, pairs_now(), allow_split_k, scratch_limit, row_gates, window_mode, pr,
                                      &launch);
  if (st != CWL_OK || !launch) return st;
  pr.p.pf_ptr = hint.ptr; pr.p.pf_bytes = hint.bytes;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
  CWL_CUDA_TRY(cudaStreamIsCapturing(stream, &capture));
  const bool capturing = capture != cudaStreamCaptureStatusNone;
  // (the entry point on the library's own scratch array, the one caller with a scratch limit, clears on every call)
  if (pr.uses_sync && (capturing || scratch_limit > 0))
    CWL_CUDA_TRY(cudaMemsetAsync(pr.ws.sync, 0, pr.ws.sync_bytes, stream));
  const cwl_status cs = configure_kernels();
  if (cs != CWL_OK) return cs;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr;
  launch_config(cfg, attr, pr.p.plan.pairs, stream, capturing);
  if (pr.p.plan.split_k > 1) CWL_CUDA_TRY(cudaLaunchKernelEx(&cfg, apply_kernel<true>, pr.maps, pr.p));
  else CWL_CUDA_TRY(cudaLaunchKernelEx(&cfg, apply_kernel<false>, pr.maps, pr.p));
  return CWL_OK;
}

// How the resident pairs are shared among the projections of a batch: in proportion to the bytes of their weights,
// at least one pair each.
void batch_shares(int n, const int* d_in, const int* d_out, int pairs, int* share) {
  double total = 0;
  for (int j = 0; j < n; ++j) total += (double)d_in[j] * d_out[j];
  int given = 0;
  for (int j = 0; j < n; ++j) {
    share[j] = (int)((double)d_in[j] * d_out[j] / total * pairs);
    if (share[j] < 1) share[j] = 1;
    given += share[j];
  }
  for (int j = 0; given < pairs; j = (j + 1) % n) { ++share[j]; ++given; }
  for (int j = 0; given > pairs; j = (j + 1) % n) if (share[j] > 1) { --share[j]; --given; }
}

cwl_status apply_impl(const void* X, int64_t ldx, const void* W, int64_t ldw, const void* A, int64_t lda,
                      const void* B, int64_t ldb, int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                      cwl_chunk_table table, int32_t window, void* Y, int64_t ldy, void* workspace,
                      size_t workspace_bytes, int32_t* status_word, void* stream, bool allow_split_k,
                      size_t scratch_limit = 0, int32_t window_mode = CWL_WINDOW_CAUSAL) {
  const bool adapter = (A != nullptr && B != nullptr && R > 0);
  cwl_projection q;
  q.W = W; q.ldw = ldw; q.A = adapter ? A : nullptr; q.lda = lda; q.B = adapter ? B : nullptr; q.ldb = ldb;
  q.Y = Y; q.ldy = ldy; q.d_out = d_out;
  return apply_group_impl(X, ldx, &q, 1, T, d_in, R, table, window, workspace, workspace_bytes, status_word, stream,
                          allow_split_k, scratch_limit, nullptr, window_mode);
}

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_apply_workspace_bytes(int32_t T, int32_t d_in, int32_t d_out, int32_t R) {
  if (T <= 0 || d_in <= 0 || d_out <= 0 || R < 0) return 256;
  cwl::ApplyWorkspace w;
  const cwl::Plan pl = cwl::make_plan(T, d_in, 1, &d_out, R, cwl::pairs_now(), true);
  return cwl::carve_apply(w, nullptr, pl, T, R);
}

extern "C" cwl_status cwl_set_pair_budget(int32_t pairs) {
  if (pairs < 0) return CWL_ERR_INVALID_ARG;
  cwl::t_pair_budget = pairs;
  return CWL_OK;
}

extern "C" cwl_status cwl_prefetch_next(const void* ptr, size_t bytes) {
  if (ptr == nullptr || bytes == 0) { cwl::t_next_prefetch = {nullptr, 0}; return CWL_OK; }
  // whole 128-byte lines inside [ptr, ptr + bytes)
  const uintptr_t lo = (reinterpret_cast<uintptr_t>(ptr) + 127u) & ~(uintptr_t)127u;
  const uintptr_t hi = (reinterpret_cast<uintptr_t>(ptr) + bytes) & ~(uintptr_t)127u;
  if (hi <= lo) { cwl::t_next_prefetch = {nullptr, 0}; return CWL_OK; }
  cwl::t_next_prefetch = {reinterpret_cast<const unsigned char*>(lo), (unsigned long long)(hi - lo)};
  return CWL_OK;
}

#ifdef CWL_TEST_HOOKS
extern "C" void cwl_debug_set(int64_t wait_limit_ns, int32_t withhold_publish) {
  cwl::g_wait_limit_ns.store(wait_limit_ns > 0 ? (unsigned long long)wait_limit_ns : cwl::kWaitLimitNs);
  cwl::g_withhold_publish.store(withhold_publish != 0 ? 1 : 0);
}

extern "C" cwl_status cwl_trace_set(long long* slots, int32_t pair) {
  if (slots == nullptr) pair = -1;
  if (cudaMemcpyToSymbol(cwl::g_trace, &slots, sizeof(slots)) != cudaSuccess) return CWL_ERR_CUDA;
  if (cudaMemcpyToSymbol(cwl::g_trace_pair, &pair, sizeof(pair)) != cudaSuccess) return CWL_ERR_CUDA;
  return CWL_OK;
}
#endif

extern "C" cwl_status cwl_apply_plan(int32_t T, int32_t d_in, int32_t d_out, int32_t R, int32_t pairs,
                                     cwl_apply_plan_info* out) {
  if (out == nullptr || T < 1 || d_in < 16 || d_out < 16 || R < 0 || pairs < 1) return CWL_ERR_INVALID_ARG;
  if (d_in % 16 != 0 || d_out % 16 != 0 || R % 16 != 0 || R > CWL_MAX_RANK) return CWL_ERR_UNSUPPORTED;
  const cwl::Plan pl = cwl::make_plan(T, d_in, 1, &d_out, R, pairs, true);
  out->pairs = pl.pairs; out->row_tiles = pl.n_m_pairs;
  out->wide_width = pl.w0; out->wide_tiles_per_row = pl.n_wide;
  out->narrow_width = pl.n_narrow > 0 ? pl.w1 : 0; out->narrow_tiles_per_row = pl.n_narrow;
  out->split_k = pl.split_k; out->k_blocks_per_split = pl.kb_per_ksplit;
  out->shrink_splits = pl.shrink_splits; out->stages = pl.stages;
  out->shrink_items = R > 0 ? pl.n_m_pairs * pl.shrink_splits : 0;
  int mx = 0, sum = 0;
  for (int g = 0; g < pl.pairs; ++g) { sum += pl.sh_count[g]; if (pl.sh_count[g] > mx) mx = pl.sh_count[g]; }
  out->shrink_items_assigned = sum; out->shrink_items_max_per_pair = mx;
  out->model_cost = pl.makespan;
  return CWL_OK;
}

extern "C" cwl_status cwl_apply(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                const void* A, int64_t lda, const void* B, int64_t ldb,
                                int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                cwl_chunk_table table, int32_t window,
                                void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                int32_t* status_word, void* stream) {
  return cwl::apply_impl(X, ldx, W, ldw, A, lda, B, ldb, T, d_in, d_out, R, table, window, Y, ldy, workspace,
                         workspace_bytes, status_word, stream, true);
}

extern "C" cwl_status cwl_apply_mode(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                     const void* A, int64_t lda, const void* B, int64_t ldb,
                                     int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                     cwl_chunk_table table, int32_t window, int32_t window_mode,
                                     void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                     int32_t* status_word, void* stream) {
  if (window_mode != CWL_WINDOW_CAUSAL && window_mode != CWL_WINDOW_CENTRED) return CWL_ERR_INVALID_ARG;
  return cwl::apply_impl(X, ldx, W, ldw, A, lda, B, ldb, T, d_in, d_out, R, table, window, Y, ldy, workspace,
                         workspace_bytes, status_word, stream, true, 0, window_mode);
}

extern "C" size_t cwl_apply_grouped_workspace_bytes(int32_t T, int32_t d_in, int32_t n_proj, const int32_t* d_out,
                                                    int32_t R) {
  if (T <= 0 || d_in <= 0 || R < 0 || d_out == nullptr || n_proj < 1 || n_proj > CWL_MAX_GROUP) return 256;
  int widths[CWL_MAX_GROUP];
  for (int j = 0; j < n_proj; ++j) { if (d_out[j] < 1) return 256; widths[j] = d_out[j]; }
  cwl::ApplyWorkspace w;
  const cwl::Plan pl = cwl::make_plan(T, d_in, n_proj, widths, R, cwl::pairs_now(), true);
  return cwl::carve_apply(w, nullptr, pl, T, R);
}

extern "C" cwl_status cwl_apply_grouped(const void* X, int64_t ldx, const cwl_projection* proj, int32_t n_proj,
                                        int32_t T, int32_t d_in, int32_t R, cwl_chunk_table table, int32_t window,
                                        void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  return cwl::apply_group_impl(X, ldx, proj, n_proj, T, d_in, R, table, window, workspace, workspace_bytes,
                               status_word, stream, true, 0);
}

extern "C" cwl_status cwl_apply_rows(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                     const void* A, int64_t lda, const void* B, int64_t ldb,
                                     int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                     const cwl_row_gate* gates, void* Y, int64_t ldy,
                                     void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  if (gates == nullptr || A == nullptr || B == nullptr || R < 1) return CWL_ERR_INVALID_ARG;
  cwl_projection q;
  q.W = W; q.ldw = ldw; q.A = A; q.lda = lda; q.B = B; q.ldb = ldb; q.Y = Y; q.ldy = ldy; q.d_out = d_out;
  cwl_chunk_table none;
  memset(&none, 0, sizeof(none));
  return cwl::apply_group_impl(X, ldx, &q, 1, T, d_in, R, none, 0, workspace, workspace_bytes, status_word, stream,
                               true, 0, gates);
}

extern "C" size_t cwl_apply_batch_workspace_bytes(int32_t T, int32_t n, const int32_t* d_in, const int32_t* d_out,
                                                  int32_t R) {
  if (T <= 0 || n < 1 || n > CWL_MAX_BATCH || d_in == nullptr || d_out == nullptr || R < 0) return 256;
  int share[CWL_MAX_BATCH];
  int di[CWL_MAX_BATCH], dn[CWL_MAX_BATCH];
  for (int j = 0; j < n; ++j) { if (d_in[j] < 1 || d_out[j] < 1) return 256; di[j] = d_in[j]; dn[j] = d_out[j]; }
  cwl::batch_shares(n, di, dn, cwl::pairs_now() < n ? n : cwl::pairs_now(), share);
  size_t total = 0;
  for (int j = 0; j < n; ++j) {
    cwl::ApplyWorkspace w;
    const cwl::Plan pl = cwl::make_plan(T, di[j], 1, &dn[j], R, share[j], true);
    total += cwl::carve_apply(w, nullptr, pl, T, R);
  }
  return total;
}

extern "C" cwl_status cwl_apply_batch(const cwl_batch_item* items, int32_t n, int32_t T, int32_t R,
                                      cwl_chunk_table table, const cwl_row_gate* gates, int32_t window,
                                      void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream_) {
  using namespace cwl;
  t_next_prefetch = {nullptr, 0};                     // a pending hint is consumed, unused
  if (items == nullptr || n < 1 || n > CWL_MAX_BATCH) return CWL_ERR_INVALID_ARG;
  const int pairs = pairs_now();
  if (pairs < n) return CWL_ERR_UNSUPPORTED;
  int di[CWL_MAX_BATCH], dn[CWL_MAX_BATCH], share[CWL_MAX_BATCH];
  for (int j = 0; j < n; ++j) {
    if (items[j].d_in < 1 || items[j].d_out < 1) return CWL_ERR_INVALID_ARG;
    di[j] = items[j].d_in; dn[j] = items[j].d_out;
  }
  batch_shares(n, di, dn, pairs, share);

  static thread_local BatchArgs args;                 // 10 KB: not on the stack of every caller
  args.n = 0;
  args.first_pair[0] = 0;
  char* ws = static_cast<char*>(workspace);
  size_t left = workspace_bytes;
  Prepared pr;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
  CWL_CUDA_TRY(cudaStreamIsCapturing(stream, &capture));
  const bool capturing = capture != cudaStreamCaptureStatusNone;
  for (int j = 0; j < n; ++j) {
    const cwl_batch_item& it = items[j];
    const bool adapter = it.A != nullptr && it.B != nullptr && R > 0;
    cwl_projection q;
    q.W = it.W; q.ldw = it.ldw; q.A = adapter ? it.A : nullptr; q.lda = it.lda; q.B = adapter ? it.B : nullptr; q.ldb = it.ldb;
    q.Y = it.Y; q.ldy = it.ldy; q.d_out = it.d_out;
    bool launch = false;
    const cwl_status st = prepare_group(it.X, it.ldx, &q, 1, T, it.d_in, R, table, window, ws, left, status_word, share[j],
                                        true, 0, gates, CWL_WINDOW_CAUSAL, pr, &launch);
    if (st != CWL_OK) return st;
    if (!launch) return CWL_OK;                       // T == 0
    ApplyWorkspace unused;
    const size_t used = carve_apply(unused, nullptr, pr.p.plan, T, pr.p.R);
    if (ws != nullptr) { ws += used; left = left >= used ? left - used : 0; }
    if (pr.uses_sync && capturing) CWL_CUDA_TRY(cudaMemsetAsync(pr.ws.sync, 0, pr.ws.sync_bytes, stream));
    const int k = args.n++;
    args.maps[k] = pr.maps;
    args.params[k] = pr.p;
    args.split[k] = pr.p.plan.split_k > 1 ? 1 : 0;
    args.first_pair[k + 1] = args.first_pair[k] + pr.p.plan.pairs;
  }
  const cwl_status cs = configure_kernels();
  if (cs != CWL_OK) return cs;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr;
  launch_config(cfg, attr, args.first_pair[args.n], stream, capturing);
  CWL_CUDA_TRY(cudaLaunchKernelEx(&cfg, apply_batch_kernel, args));
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

extern "C" size_t cwl_apply_noalloc_scratch_need(int32_t T, int32_t d_in, int32_t d_out, int32_t R) {
  if (T <= 0 || d_in <= 0 || d_out <= 0 || R < 0) return 256;
  cwl::ApplyWorkspace w;
  const cwl::Plan pl = cwl::make_plan(T, d_in, 1, &d_out, R, cwl::pairs_now(), false, CWL_NOALLOC_SCRATCH_BYTES);
  return cwl::carve_apply(w, nullptr, pl, T, R);
}

extern "C" cwl_status cwl_apply_noalloc(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                        const void* A, int64_t lda, const void* B, int64_t ldb,
                                        int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                                        cwl_chunk_table table, int32_t window,
                                        void* Y, int64_t ldy, int32_t* status_word, void* stream) {
  if (T < 0 || d_in < 1 || d_out < 1 || R < 0) return CWL_ERR_INVALID_ARG;
  const bool adapter = (A != nullptr && B != nullptr && R > 0);
  {
    // the same argument checks, in the same order, as cwl_apply makes: a bad shape is reported as such, not as a
    // scratch problem
    cwl_projection q;
    q.W = W; q.ldw = ldw; q.A = adapter ? A : nullptr; q.lda = lda; q.B = adapter ? B : nullptr; q.ldb = ldb;
    q.Y = Y; q.ldy = ldy; q.d_out = d_out;
    bool with_adapter = false;
    const cwl_status chk = cwl::check_group(X, ldx, &q, 1, T, d_in, R, table, nullptr, window, with_adapter);
    if (chk != CWL_OK) return chk;
  }
  if (adapter && T > 0 && cwl_apply_noalloc_scratch_need(T, d_in, d_out, R) > (size_t)CWL_NOALLOC_SCRATCH_BYTES)
    return CWL_ERR_WORKSPACE;  // the problem needs more scratch than the built-in array holds
  void* scratch = nullptr;
  const cwl_status st = cwl::noalloc_scratch(&scratch);
  if (st != CWL_OK) return st;
  // every tile keeps its whole K loop here: the partial accumulators of a split K loop would not fit
  return cwl::apply_impl(X, ldx, W, ldw, A, lda, B, ldb, T, d_in, d_out, R, table, window, Y, ldy, scratch,
                         (size_t)CWL_NOALLOC_SCRATCH_BYTES, status_word, stream, false, CWL_NOALLOC_SCRATCH_BYTES);
}
