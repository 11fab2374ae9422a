// cwl_batch_align: batch alignment (Sec. III-G, IV-F).  Sequences of a batch are bucketed by complexity
// percentile; the members of a bucket share their chunk joins, worked out once on the bucket's pooled score
// track; rung, budget, rank and scale stay per sequence (Sec. III-C).
//
// Passes (all comparisons are integer, so the result is a function of the fp32 scores only):
//   1. quantise to Q24 and prefix sums P over the packed scores                       (as in cwl_partition)
//   2. per sequence: its position in the complexity order (mean = sum / len compared by cross-multiplication,
//      lower index first on ties, empty sequences first) and its bucket               (one thread per sequence)
//   3. per bucket: the longest member; the buckets' tracks laid out one after another (one block)
//   4. pooled track: S[j] += q, N[j] += 1 at the token's position inside its sequence (one thread per token,
//      integer atomics: the order of the additions cannot matter)
//   5. prefix sums of S and N inside every bucket's track                             (one block per bucket)
//   6. the greedy walk of Sec. III-B on each pooled track                             (one warp per bucket,
//      32 candidate cuts at a time)
//   7. per sequence: which of its bucket's joins it takes, its chunks' rungs from its own P, the budget,
//      compaction into the caller's table                                             (one block per sequence)
#include "partition_common.cuh"

namespace cwl {
namespace {

constexpr int kAlignThreads = 256;
constexpr int kMaxBuckets = 1024;
constexpr int kMaxAlignT = 1 << 19;     // keeps every cross product sum * len below 2^62

struct AlignWorkspace {
  int64_t* P;            // [T + 1]
  int64_t* tile_sum;     // [n_tiles]
  int64_t* PS;           // [T + n_buckets + 1] pooled sums, then their prefix sums; bucket k at [base[k], base[k] + L_k]
  int32_t* PN;           // same layout: members present at a position, then prefix sums
  int32_t* base;         // [n_buckets + 1]
  int32_t* blen;         // [n_buckets] longest member of each bucket
  int32_t* joins;        // [T + n_buckets + 1] shared joins of bucket k at [base[k], base[k] + n_joins[k])
  int32_t* n_joins;      // [n_buckets]
  int32_t* count;        // [n_seq] chunks per sequence
  int32_t* rung0;        // [T] rung of a sequence's chunks as cut, at [cu[n], cu[n] + count[n])
  size_t pooled_entries;
};

inline size_t carve_align(AlignWorkspace& w, char* base, int32_t T, int32_t n_seq, int32_t n_buckets) {
  size_t off = 0;
  const size_t Tn = (size_t)(T > 0 ? T : 1), n_tiles = (size_t)ceil_div64(Tn, kScanTile);
  const size_t pooled = Tn + (size_t)n_buckets + 1;
  auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off = align_up(off + bytes, 16); return p; };
  w.P = reinterpret_cast<int64_t*>(take(sizeof(int64_t) * (Tn + 1)));
  w.tile_sum = reinterpret_cast<int64_t*>(take(sizeof(int64_t) * n_tiles));
  w.PS = reinterpret_cast<int64_t*>(take(sizeof(int64_t) * pooled));
  w.PN = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * pooled));
  w.base = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * ((size_t)n_buckets + 1)));
  w.blen = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)n_buckets));
  w.joins = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * pooled));
  w.n_joins = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)n_buckets));
  w.count = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(n_seq > 0 ? n_seq : 1)));
  w.rung0 = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * Tn));
  w.pooled_entries = pooled;
  return off;
}

// pass 2: position in the complexity order and percentile bucket of every sequence
__global__ void __launch_bounds__(kAlignThreads)
seq_order_kernel(const int64_t* __restrict__ P, const int32_t* __restrict__ cu, int n_seq, int n_buckets,
                 int32_t* __restrict__ order_pos, int32_t* __restrict__ bucket) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= n_seq) return;
  const int64_t len_n = cu[n + 1] - cu[n], sum_n = P[cu[n + 1]] - P[cu[n]];
  int before = 0;
  for (int m = 0; m < n_seq; ++m) {
    if (m == n) continue;
    const int64_t len_m = cu[m + 1] - cu[m];
    bool m_first;
    if (len_m == 0 || len_n == 0) {
      m_first = (len_m == 0 && len_n == 0) ? (m < n) : (len_m == 0);
    } else {
      const int64_t lhs = (P[cu[m + 1]] - P[cu[m]]) * len_n, rhs = sum_n * len_m;   // mean_m against mean_n
      m_first = lhs < rhs || (lhs == rhs && m < n);
    }
    before += m_first ? 1 : 0;
  }
  order_pos[n] = before;
  bucket[n] = (int32_t)(((int64_t)before * n_buckets) / n_seq);
}

// pass 3: longest member per bucket and where each bucket's pooled track starts (L_k + 1 entries each)
__global__ void __launch_bounds__(kMaxBuckets)
bucket_layout_kernel(const int32_t* __restrict__ cu, const int32_t* __restrict__ bucket, int n_seq, int n_buckets,
                     int32_t* __restrict__ blen, int32_t* __restrict__ base) {
  __shared__ int32_t len_s[kMaxBuckets];
  const int k = threadIdx.x;
  if (k < n_buckets) {
    int L = 0;
    for (int n = 0; n < n_seq; ++n)
      if (bucket[n] == k) L = max(L, cu[n + 1] - cu[n]);
    len_s[k] = L;
    blen[k] = L;
  }
  __syncthreads();
  if (k == 0) {
    int run = 0;
    for (int i = 0; i < n_buckets; ++i) { base[i] = run; run += len_s[i] + 1; }
    base[n_buckets] = run;
  }
}

// pass 4: pooled track (integer atomics; PS and PN were cleared before)
__global__ void __launch_bounds__(kAlignThreads)
pool_kernel(const float* __restrict__ score, const int32_t* __restrict__ cu, int n_seq, int T,
            const int32_t* __restrict__ bucket, const int32_t* __restrict__ base,
            unsigned long long* __restrict__ S, int32_t* __restrict__ N) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  int lo = 0, hi = n_seq;                // cu[lo] <= t < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  const int at = base[bucket[lo]] + (t - cu[lo]);
  atomicAdd(S + at, (unsigned long long)quantise(score[t]));
  atomicAdd(N + at, 1);
}

// pass 5: exclusive prefix sums of a bucket's track, in place, over its L_k + 1 entries (the last one receives the total)
__global__ void __launch_bounds__(kAlignThreads)
pooled_prefix_kernel(const int32_t* __restrict__ base, const int32_t* __restrict__ blen,
                     int64_t* __restrict__ PS, int32_t* __restrict__ PN) {
  __shared__ int64_t tot_s[kAlignThreads];
  __shared__ int64_t tot_n[kAlignThreads];
  const int k = blockIdx.x, tid = threadIdx.x;
  const int L = blen[k], b0 = base[k];
  const int per = ceil_div(L + 1, kAlignThreads);
  const int lo = min(L + 1, tid * per), hi = min(L + 1, lo + per);
  int64_t s = 0, c = 0;
  for (int j = lo; j < hi; ++j) { s += (j < L) ? PS[b0 + j] : 0; c += (j < L) ? PN[b0 + j] : 0; }
  tot_s[tid] = s; tot_n[tid] = c;
  __syncthreads();
  int64_t run_s = 0, run_n = 0;
  for (int i = 0; i < tid; ++i) { run_s += tot_s[i]; run_n += tot_n[i]; }
  for (int j = lo; j < hi; ++j) {
    const int64_t vs = (j < L) ? PS[b0 + j] : 0;
    const int32_t vn = (j < L) ? PN[b0 + j] : 0;
    PS[b0 + j] = run_s; PN[b0 + j] = (int32_t)run_n;
    run_s += vs; run_n += vn;
  }
}

// pass 6: the walk of Sec. III-B on the pooled track of bucket k = blockIdx.x (one warp)
__global__ void __launch_bounds__(32)
pooled_walk_kernel(const int32_t* __restrict__ base, const int32_t* __restrict__ blen, Ladder Ld,
                   const int64_t* __restrict__ PS, const int32_t* __restrict__ PN,
                   int32_t* __restrict__ joins, int32_t* __restrict__ n_joins) {
  const int k = blockIdx.x, lane = threadIdx.x;
  const int L = blen[k], b0 = base[k];
  const int64_t* ps = PS + b0;
  const int32_t* pn = PN + b0;
  int nj = 0, b = 0;
  while (b < L) {
    int cut = L;
    if (L - b >= 2 * Ld.min_len) {
      const int first = b + Ld.min_len;
      const int last = min(L - Ld.min_len, b + Ld.max_len);        // the candidate at b + max_len always stops
      const int64_t sb = ps[b];
      const int32_t nb = pn[b];
      for (int e0 = first; e0 <= last && cut == L; e0 += 32) {
        const int e = e0 + lane;
        bool stop = false;
        if (e <= last) {
          if (e - b >= Ld.max_len) stop = true;
          else {
            const int64_t se = ps[e];
            const int32_t ne = pn[e];
            stop = rung_of(se - sb, (int64_t)(ne - nb), Ld) !=
                   rung_of(ps[e + Ld.min_len] - se, (int64_t)(pn[e + Ld.min_len] - ne), Ld);
          }
        }
        const unsigned m = __ballot_sync(0xffffffffu, stop);
        if (m != 0) cut = e0 + __ffs(m) - 1;
      }
    }
    if (cut < L) { if (lane == 0) joins[b0 + nj] = cut; ++nj; }
    b = cut;
  }
  if (lane == 0) n_joins[k] = nj;
}

// pass 7a: chunks of every sequence = 1 + the joins of its bucket that leave it at least min_len tokens
__global__ void __launch_bounds__(kAlignThreads)
member_count_kernel(const int32_t* __restrict__ cu, const int32_t* __restrict__ bucket, int n_seq, int min_len,
                    const int32_t* __restrict__ base, const int32_t* __restrict__ joins,
                    const int32_t* __restrict__ n_joins, int32_t* __restrict__ count) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= n_seq) return;
  const int len = cu[n + 1] - cu[n];
  if (len == 0) { count[n] = 0; return; }
  const int k = bucket[n], nj = n_joins[k];
  const int32_t* jk = joins + base[k];
  int lo = 0, hi = nj;                   // joins ascend: first index whose join exceeds len - min_len
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (jk[mid] <= len - min_len) lo = mid + 1; else hi = mid;
  }
  count[n] = lo + 1;
}

// pass 7b: the sequence's chunks into the caller's table: own rungs, budget, rank and scale
__global__ void __launch_bounds__(kAlignThreads)
emit_aligned_kernel(const int64_t* __restrict__ P, const int32_t* __restrict__ cu, const int32_t* __restrict__ bucket,
                    int n_seq, int T, Ladder Ld, const int32_t* __restrict__ base, const int32_t* __restrict__ joins,
                    const int32_t* __restrict__ count, int32_t* __restrict__ rung0, cwl_chunk_table table,
                    int32_t* status_word) {
  __shared__ int64_t red[32];
  const int n = blockIdx.x, tid = threadIdx.x;
  int64_t before = 0;
  for (int i = tid; i < n && i < n_seq; i += blockDim.x) before += count[i];
  const int first = (int)block_sum64(before, red);
  const int C = (n < n_seq) ? count[n] : 0;
  const bool fits = (int64_t)first + C <= (int64_t)table.capacity;
  if (n < n_seq && fits && C > 0) {
    const int S = cu[n], len = cu[n + 1] - cu[n];
    const int32_t* jk = joins + base[bucket[n]];
    auto start_of = [&](int c) { return c == 0 ? 0 : jk[c - 1]; };
    auto end_of = [&](int c) { return c == C - 1 ? len : jk[c]; };
    for (int c = tid; c < C; c += blockDim.x)
      rung0[S + c] = rung_of(P[S + end_of(c)] - P[S + start_of(c)], end_of(c) - start_of(c), Ld);
    __syncthreads();
    const int top = Ld.n_rungs - 1;
    for (int c = tid; c < C; c += blockDim.x) {
      int r = rung0[S + c];
      if (Ld.hi_budget >= 0 && Ld.n_rungs >= 2 && r == top) {
        // keeps the top rung only if fewer than hi_budget top-rung chunks of the sequence have a larger mean
        const int64_t len_c = end_of(c) - start_of(c), sum_c = P[S + end_of(c)] - P[S + start_of(c)];
        int better = 0;
        for (int d = 0; d < C; ++d) {
          if (d == c || rung0[S + d] != top) continue;
          const int64_t len_d = end_of(d) - start_of(d);
          const int64_t lhs = (P[S + end_of(d)] - P[S + start_of(d)]) * len_c, rhs = sum_c * len_d;
          if (lhs > rhs || (lhs == rhs && d < c)) ++better;
        }
        if (better >= Ld.hi_budget) r = top - 1;
      }
      table.offsets[first + c] = S + start_of(c);
      table.rung[first + c] = r;
      table.rank[first + c] = Ld.rung_rank[r];
      table.scale[first + c] = Ld.rung_scale[r];
      table.flags[first + c] = (c == 0) ? 1 : 0;
    }
  }
  if (n == max(n_seq, 1) - 1 && tid == 0) {      // the last block owns the totals
    if (fits) {
      table.offsets[first + C] = T;
      *table.n_chunks = first + C;
    } else {
      *table.n_chunks = 0;
      flag_status(status_word, CWL_ERR_CAPACITY);
    }
  }
}

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_batch_align_workspace_bytes(int32_t T, int32_t n_seq, int32_t n_buckets) {
  if (T < 0 || n_seq < 0 || n_buckets < 1) return 0;
  cwl::AlignWorkspace w;
  return cwl::carve_align(w, nullptr, T, n_seq, n_buckets);
}

extern "C" cwl_status cwl_batch_align(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                                      const cwl_policy* policy, int32_t n_buckets, cwl_chunk_table table,
                                      int32_t* bucket, int32_t* order_pos,
                                      void* workspace, size_t workspace_bytes,
                                      int32_t* status_word, void* stream_) {
  using namespace cwl;
  if (T < 0 || n_seq < 0 || n_buckets < 1 || cu_seqlens == nullptr || (score == nullptr && T > 0))
    return CWL_ERR_INVALID_ARG;
  if (!policy_ok(policy)) return CWL_ERR_INVALID_ARG;
  if (table.offsets == nullptr || table.rank == nullptr || table.scale == nullptr || table.rung == nullptr ||
      table.flags == nullptr || table.n_chunks == nullptr || table.capacity < 0)
    return CWL_ERR_INVALID_ARG;
  if (n_seq > 0 && (bucket == nullptr || order_pos == nullptr)) return CWL_ERR_INVALID_ARG;
  if (T > 0 && n_seq == 0) return CWL_ERR_INVALID_ARG;
  if (T > kMaxAlignT || n_buckets > kMaxBuckets) return CWL_ERR_UNSUPPORTED;
  AlignWorkspace w;
  const size_t need = carve_align(w, static_cast<char*>(workspace), T, n_seq, n_buckets);
  if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return CWL_ERR_WORKSPACE;
  const Ladder L = make_ladder(policy);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int seq_blocks = n_seq > 0 ? ceil_div(n_seq, kAlignThreads) : 1;

  if (T > 0) {
    const int n_tiles = (int)ceil_div64(T, kScanTile);
    const bool few_tiles = n_tiles <= 32;
    if (!few_tiles) tile_sum_kernel<<<n_tiles, kScanThreads, 0, stream>>>(score, T, w.tile_sum);
    prefix_kernel<<<n_tiles, kScanThreads, 0, stream>>>(score, T, few_tiles ? (const int64_t*)nullptr : (const int64_t*)w.tile_sum, w.P);
  } else {
    CWL_CUDA_TRY(cudaMemsetAsync(w.P, 0, sizeof(int64_t), stream));
  }
  if (n_seq > 0) {
    seq_order_kernel<<<seq_blocks, kAlignThreads, 0, stream>>>(w.P, cu_seqlens, n_seq, n_buckets, order_pos, bucket);
    bucket_layout_kernel<<<1, kMaxBuckets, 0, stream>>>(cu_seqlens, bucket, n_seq, n_buckets, w.blen, w.base);
    CWL_CUDA_TRY(cudaMemsetAsync(w.PS, 0, sizeof(int64_t) * w.pooled_entries, stream));
    CWL_CUDA_TRY(cudaMemsetAsync(w.PN, 0, sizeof(int32_t) * w.pooled_entries, stream));
    if (T > 0)
      pool_kernel<<<ceil_div(T, kAlignThreads), kAlignThreads, 0, stream>>>(
          score, cu_seqlens, n_seq, T, bucket, w.base, reinterpret_cast<unsigned long long*>(w.PS), w.PN);
    pooled_prefix_kernel<<<n_buckets, kAlignThreads, 0, stream>>>(w.base, w.blen, w.PS, w.PN);
    pooled_walk_kernel<<<n_buckets, 32, 0, stream>>>(w.base, w.blen, L, w.PS, w.PN, w.joins, w.n_joins);
    member_count_kernel<<<seq_blocks, kAlignThreads, 0, stream>>>(cu_seqlens, bucket, n_seq, L.min_len, w.base, w.joins,
                                                                 w.n_joins, w.count);
  }
  emit_aligned_kernel<<<n_seq > 0 ? n_seq : 1, kAlignThreads, 0, stream>>>(
      w.P, cu_seqlens, bucket, n_seq, T, L, w.base, w.joins, w.count, w.rung0, table, status_word);
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
}
