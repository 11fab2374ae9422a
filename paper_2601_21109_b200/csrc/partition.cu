// cwl_partition: adaptive chunker (Sec. III-B) and rank-ladder selector (Sec. III-C).
//
// The greedy walk is chunk-sequential, but the cut that follows a chunk start b depends on b
// alone.  So the work is split into data-parallel passes and one short pointer chase:
//   1. quantise scores to Q24 integers and reduce per tile            (grid over T)
//   2. exclusive prefix sums P[0..T] (int64)                          (grid over T)
//   3. next_cut[b] for EVERY position b: first stopping candidate     (one warp per b, ballot)
//   4. per sequence: chase next_cut from the sequence start through shared memory, then
//      rung per chunk and the high-capacity budget                    (one block per sequence)
//   5. compact the per-sequence lists into the caller's chunk table   (one block per sequence)
// All comparisons are integer, so the table is a function of the fp32 scores only.
#include "partition_common.cuh"

namespace cwl {
namespace {

constexpr int kWalkThreads = 256;
constexpr int kCutUnroll = 4;         // candidate cuts per lane and round in pass 3
constexpr int kWalkSegment = 8192;                    // next_cut entries staged per shared-memory segment

struct Workspace {
  int64_t* P;          // [T + 1]
  int64_t* tile_sum;   // [n_tiles]
  int32_t* next_cut;   // [T]
  int32_t* seq_start;  // [T] chunk starts of sequence n live at [cu[n], cu[n] + count[n])
  int32_t* seq_rung0;  // [T] rung as walked
  int32_t* seq_rung;   // [T] rung after the budget
  int32_t* count;      // [n_seq]
};

inline size_t carve(Workspace& w, char* base, int32_t T, int32_t n_seq) {
  size_t off = 0;
  const size_t n_tiles = (size_t)ceil_div64(T > 0 ? T : 1, kScanTile);
  auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off = align_up(off + bytes, 16); return p; };
  w.P = reinterpret_cast<int64_t*>(take(sizeof(int64_t) * ((size_t)T + 1)));
  w.tile_sum = reinterpret_cast<int64_t*>(take(sizeof(int64_t) * n_tiles));
  w.next_cut = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(T > 0 ? T : 1)));
  w.seq_start = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(T > 0 ? T : 1)));
  w.seq_rung0 = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(T > 0 ? T : 1)));
  w.seq_rung = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(T > 0 ? T : 1)));
  w.count = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (size_t)(n_seq > 0 ? n_seq : 1)));
  return off;
}

// pass 3: the cut that closes a chunk opened at b (one warp per b)
__global__ void __launch_bounds__(256)
next_cut_kernel(const int64_t* __restrict__ P, const int32_t* __restrict__ cu, int n_seq, int T,
                Ladder L, int32_t* __restrict__ next_cut) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int64_t b64 = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); b64 < T;
       b64 += (int64_t)gridDim.x * warps_per_block) {
    const int b = (int)b64;
    // sequence of b: last n with cu[n] <= b (skips empty sequences)
    int lo = 0, hi = n_seq;  // invariant: cu[lo] <= b < cu[hi]
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (cu[mid] <= b) lo = mid; else hi = mid;
    }
    const int E = cu[lo + 1];
    int cut = E;
    if (E - b >= 2 * L.min_len) {
      const int first = b + L.min_len;
      const int last = min(E - L.min_len, b + L.max_len);  // the candidate at b + max_len always stops
      const int64_t Pb = P[b];
      // kCutUnroll x 32 candidates per round, all their loads in flight together (a round is a chain of dependent
      // L2 accesses, and most chunks close within the first hundred candidates)
      for (int base = first; base <= last && cut == E; base += 32 * kCutUnroll) {
        bool stop[kCutUnroll];
#pragma unroll
        for (int u = 0; u < kCutUnroll; ++u) {
          const int e = base + u * 32 + lane;
          stop[u] = false;
          if (e <= last) {
            if (e - b >= L.max_len) {
              stop[u] = true;
            } else {
              const int64_t Pe = P[e];
              stop[u] = rung_of(Pe - Pb, e - b, L) != rung_of(P[e + L.min_len] - Pe, L.min_len, L);
            }
          }
        }
#pragma unroll
        for (int u = 0; u < kCutUnroll; ++u) {
          const unsigned m = __ballot_sync(0xffffffffu, stop[u]);
          if (m != 0 && cut == E) cut = base + u * 32 + __ffs(m) - 1;
        }
      }
    }
    if (lane == 0) next_cut[b] = cut;
  }
}

// pass 4: chase the cuts of one sequence, then rung and budget per chunk
__global__ void __launch_bounds__(kWalkThreads)
walk_kernel(const int64_t* __restrict__ P, const int32_t* __restrict__ cu, Ladder L,
            const int32_t* __restrict__ next_cut, int32_t* __restrict__ seq_start,
            int32_t* __restrict__ seq_rung0, int32_t* __restrict__ seq_rung, int32_t* __restrict__ count,
            bool emit_here, int T, cwl_chunk_table table, int32_t* status_word) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int32_t seg[kWalkSegment];
  __shared__ int s_pos, s_count;
  const int n = blockIdx.x, tid = threadIdx.x;
  const int S = cu[n], E = cu[n + 1];
  if (tid == 0) { s_pos = S; s_count = 0; }
  __syncthreads();
  while (true) {
    const int seg_base = s_pos;
    if (seg_base >= E) break;
    const int seg_end = min(E, seg_base + kWalkSegment);
    for (int i = seg_base + tid; i < seg_end; i += kWalkThreads) seg[i - seg_base] = next_cut[i];
    __syncthreads();
    if (tid == 0) {
      int b = seg_base, c = s_count;
      while (b < seg_end) {
        seq_start[S + c] = b;   // chunks are non-empty, so a sequence never has more chunks than tokens
        ++c;
        b = seg[b - seg_base];
      }
      s_pos = b;
      s_count = c;
    }
    __syncthreads();
  }
  const int C = s_count;
  if (tid == 0) count[n] = C;
  // rung of every chunk as walked
  for (int c = tid; c < C; c += kWalkThreads) {
    const int b = seq_start[S + c], e = (c + 1 < C) ? seq_start[S + c + 1] : E;
    const int r = rung_of(P[e] - P[b], e - b, L);
    seq_rung0[S + c] = r;
    seq_rung[S + c] = r;
  }
  __syncthreads();
  // budget on high-capacity regions: a top-rung chunk keeps its rung only if fewer than
  // hi_budget top-rung chunks of this sequence have a larger mean (earlier chunk wins ties)
  const int top = L.n_rungs - 1;
  for (int c = tid; c < C && L.hi_budget >= 0 && L.n_rungs >= 2; c += kWalkThreads) {
    if (seq_rung0[S + c] != top) continue;
    const int bc = seq_start[S + c], ec = (c + 1 < C) ? seq_start[S + c + 1] : E;
    const int64_t sum_c = P[ec] - P[bc], len_c = ec - bc;
    int better = 0;
    for (int d = 0; d < C; ++d) {
      if (d == c || seq_rung0[S + d] != top) continue;
      const int bd = seq_start[S + d], ed = (d + 1 < C) ? seq_start[S + d + 1] : E;
      const int64_t lhs = (P[ed] - P[bd]) * len_c, rhs = sum_c * (int64_t)(ed - bd);
      if (lhs > rhs || (lhs == rhs && d < c)) ++better;
    }
    if (better >= L.hi_budget) seq_rung[S + c] = top - 1;
  }
  if (!emit_here) return;
  // a single sequence: this block is the only one, and writes the caller's table itself (pass 5 is not launched)
  __syncthreads();
  const bool fits = C <= table.capacity;
  for (int c = tid; c < C && fits; c += kWalkThreads) {
    const int r = seq_rung[S + c];
    table.offsets[c] = seq_start[S + c];
    table.rung[c] = r;
    table.rank[c] = L.rung_rank[r];
    table.scale[c] = L.rung_scale[r];
    table.flags[c] = (c == 0) ? 1 : 0;
  }
  if (tid == 0) {
    if (fits) {
      table.offsets[C] = T;
      *table.n_chunks = C;
    } else {
      *table.n_chunks = 0;
      flag_status(status_word, CWL_ERR_CAPACITY);
    }
  }
}

// pass 5: compaction into the caller's table
__global__ void __launch_bounds__(256)
emit_kernel(const int32_t* __restrict__ cu, int n_seq, int T, Ladder L,
            const int32_t* __restrict__ seq_start, const int32_t* __restrict__ seq_rung,
            const int32_t* __restrict__ count, cwl_chunk_table table, int32_t* status_word) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int64_t red[32];
  const int n = blockIdx.x, tid = threadIdx.x;
  int64_t before = 0;
  for (int i = tid; i < n && i < n_seq; i += blockDim.x) before += count[i];
  const int base = (int)block_sum64(before, red);
  const int C = (n < n_seq) ? count[n] : 0;
  const bool fits = (int64_t)base + C <= (int64_t)table.capacity;
  if (n < n_seq && fits) {
    const int S = cu[n];
    for (int c = tid; c < C; c += blockDim.x) {
      const int r = seq_rung[S + c];
      table.offsets[base + c] = seq_start[S + c];
      table.rung[base + c] = r;
      table.rank[base + c] = L.rung_rank[r];
      table.scale[base + c] = L.rung_scale[r];
      table.flags[base + c] = (c == 0) ? 1 : 0;
    }
  }
  if (n == max(n_seq, 1) - 1 && tid == 0) {  // the last block owns the totals
    if (fits) {
      table.offsets[base + C] = T;
      *table.n_chunks = base + C;
    } else {
      *table.n_chunks = 0;
      flag_status(status_word, CWL_ERR_CAPACITY);
    }
  }
}

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_partition_workspace_bytes(int32_t T, int32_t n_seq) {
  if (T < 0 || n_seq < 0) return 0;
  cwl::Workspace w;
  return cwl::carve(w, nullptr, T, n_seq);
}

extern "C" cwl_status cwl_partition(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                                    const cwl_policy* policy, cwl_chunk_table table,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status_word, void* stream_) {
  using namespace cwl;
  if (T < 0 || n_seq < 0 || cu_seqlens == nullptr || (score == nullptr && T > 0)) return CWL_ERR_INVALID_ARG;
  if (!policy_ok(policy)) return CWL_ERR_INVALID_ARG;
  if (table.offsets == nullptr || table.rank == nullptr || table.scale == nullptr || table.rung == nullptr ||
      table.flags == nullptr || table.n_chunks == nullptr || table.capacity < 0)
    return CWL_ERR_INVALID_ARG;
  if (T > 0 && n_seq == 0) return CWL_ERR_INVALID_ARG;
  Workspace w;
  const size_t need = carve(w, static_cast<char*>(workspace), T, n_seq);
  if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return CWL_ERR_WORKSPACE;

  const Ladder L = make_ladder(policy);

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const bool chained = !stream_is_capturing(stream);   // each kernel waits for the one before it by itself
  bool emitted = false;
  if (T > 0) {
    const int n_tiles = (int)ceil_div64(T, kScanTile);
    const bool few_tiles = n_tiles <= 32;                // then pass 2 adds up the scores before its tile itself
    if (!few_tiles)
      CWL_CUDA_TRY(launch_chained(chained, tile_sum_kernel, dim3(n_tiles), dim3(kScanThreads), 0, stream, score, T, w.tile_sum));
    CWL_CUDA_TRY(launch_chained(chained, prefix_kernel, dim3(n_tiles), dim3(kScanThreads), 0, stream, score, T,
                                few_tiles ? (const int64_t*)nullptr : (const int64_t*)w.tile_sum, w.P));
    const int warps_per_block = 8;
    int64_t blocks = ceil_div64(T, warps_per_block);
    if (blocks > 148 * 64) blocks = 148 * 64;
    CWL_CUDA_TRY(launch_chained(chained, next_cut_kernel, dim3((int)blocks), dim3(warps_per_block * 32), 0, stream, w.P,
                                cu_seqlens, n_seq, T, L, w.next_cut));
    emitted = n_seq == 1;                                // one sequence: pass 4 writes the table too
    CWL_CUDA_TRY(launch_chained(chained, walk_kernel, dim3(n_seq), dim3(kWalkThreads), 0, stream, w.P, cu_seqlens, L,
                                w.next_cut, w.seq_start, w.seq_rung0, w.seq_rung, w.count, emitted, T, table, status_word));
  } else if (n_seq > 0) {
    CWL_CUDA_TRY(cudaMemsetAsync(w.count, 0, sizeof(int32_t) * (size_t)n_seq, stream));
  }
  if (!emitted)
    CWL_CUDA_TRY(launch_chained(chained && T > 0, emit_kernel, dim3(n_seq > 0 ? n_seq : 1), dim3(256), 0, stream, cu_seqlens,
                                n_seq, T, L, w.seq_start, w.seq_rung, w.count, table, status_word));
  return CWL_OK;
}
