// Pieces shared by the chunker (partition.cu) and the batch aligner (align.cu): the Q24 fixed point of Sec. III-B's
// chunk means, the rung rule of Sec. III-C, the prefix-sum passes and the policy checks.  Everything lives in an
// unnamed namespace, so each translation unit has its own copy.
#pragma once

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;  // scores per block in passes 1 and 2

struct Ladder {
  int32_t n_rungs;
  int32_t min_len, max_len, hi_budget;
  int64_t theta_q[CWL_MAX_RUNGS - 1];  // floor(threshold * 2^24)
  int32_t rung_rank[CWL_MAX_RUNGS];
  float rung_scale[CWL_MAX_RUNGS];
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ int32_t quantise(float s) {
  if (s != s) return kQ24;  // NaN: hardest
  s = fminf(fmaxf(s, 0.f), 1.f);
  return __float2int_rd(s * 16777216.0f);  // exact: power-of-two scaling, then floor
}

__device__ __forceinline__ int rung_of(int64_t sum, int64_t len, const Ladder& L) {
  int k = 0;
#pragma unroll
  for (int j = 0; j < CWL_MAX_RUNGS - 1; ++j)
    if (j + 1 < L.n_rungs && sum >= L.theta_q[j] * len) ++k;
  return k;
}

__device__ __forceinline__ int64_t warp_sum64(int64_t v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// Block-wide sum of one int64 per thread; result valid in every thread.
__device__ int64_t block_sum64(int64_t v, int64_t* smem /* >= 32 entries */) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum64(v);
  __syncthreads();
  if (lane == 0) smem[wid] = v;
  __syncthreads();
  int64_t t = (lane < nw) ? smem[lane] : 0;
  return warp_sum64(t);
}

// pass 1: per-tile sums of quantised scores
__global__ void __launch_bounds__(kScanThreads)
tile_sum_kernel(const float* __restrict__ score, int T, int64_t* __restrict__ tile_sum) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int64_t red[32];
  const int base = blockIdx.x * kScanTile;
  int64_t s = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    int t = base + i * kScanThreads + threadIdx.x;
    if (t < T) s += quantise(score[t]);
  }
  s = block_sum64(s, red);
  if (threadIdx.x == 0) tile_sum[blockIdx.x] = s;
}

// pass 2: exclusive prefix sums.  Each block adds up the tiles before it, then scans its own.  With tile_sum == NULL
// (a few tiles only: pass 1 is not worth a launch) it adds up the scores before its tile itself; the sums are
// integers, so the result is the same bit for bit.
__global__ void __launch_bounds__(kScanThreads)
prefix_kernel(const float* __restrict__ score, int T, const int64_t* __restrict__ tile_sum,
              int64_t* __restrict__ P) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ int64_t red[32];
  __shared__ int64_t warp_tot[kScanThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int64_t before = 0;
  if (tile_sum != nullptr) {
    for (int i = tid; i < (int)blockIdx.x; i += kScanThreads) before += tile_sum[i];
  } else {
    for (int t = tid; t < (int)blockIdx.x * kScanTile; t += kScanThreads) before += quantise(score[t]);
  }
  before = block_sum64(before, red);

  // thread-contiguous items: thread tid owns [base + tid*kScanItems, +kScanItems)
  const int t0 = blockIdx.x * kScanTile + tid * kScanItems;
  int32_t q[kScanItems];
  int64_t mine = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    q[i] = (t0 + i < T) ? quantise(score[t0 + i]) : 0;
    mine += q[i];
  }
  int64_t incl = mine;  // inclusive warp scan of per-thread totals
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    int64_t o = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += o;
  }
  if (lane == 31) warp_tot[wid] = incl;
  __syncthreads();
  int64_t warp_before = 0;
  for (int w = 0; w < wid; ++w) warp_before += warp_tot[w];
  int64_t run = before + warp_before + (incl - mine);
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    if (t0 + i < T) P[t0 + i] = run;
    run += q[i];
    if (t0 + i == T - 1) P[T] = run;
  }
  if (T == 0 && blockIdx.x == 0 && tid == 0) P[0] = 0;
}

bool policy_ok(const cwl_policy* p) {
  if (p == nullptr || p->n_rungs < 1 || p->n_rungs > CWL_MAX_RUNGS) return false;
  if (p->min_len < 1 || p->max_len < p->min_len) return false;
  if ((int64_t)p->min_len + (int64_t)p->max_len > (int64_t)(1 << 19)) return false;
  if (p->window < 0 || p->window > p->min_len) return false;
  for (int k = 0; k < p->n_rungs; ++k) {
    if (p->rung_rank[k] < 0 || p->rung_rank[k] > CWL_MAX_RANK) return false;
    if (k > 0 && p->rung_rank[k] < p->rung_rank[k - 1]) return false;
  }
  for (int k = 0; k + 1 < p->n_rungs; ++k) {
    const float th = p->threshold[k];
    if (!(th >= 0.f && th <= 1.f)) return false;
    if (k > 0 && !(th > p->threshold[k - 1])) return false;
  }
  return true;
}


// the policy in the form the kernels take: thresholds in Q24, ladder by value
inline Ladder make_ladder(const cwl_policy* policy) {
  Ladder L{};
  L.n_rungs = policy->n_rungs;
  L.min_len = policy->min_len;
  L.max_len = policy->max_len;
  L.hi_budget = policy->hi_budget;
  for (int k = 0; k < policy->n_rungs; ++k) {
    L.rung_rank[k] = policy->rung_rank[k];
    L.rung_scale[k] = policy->rung_scale[k];
  }
  for (int k = 0; k + 1 < policy->n_rungs; ++k)
    L.theta_q[k] = (int64_t)__builtin_floor((double)policy->threshold[k] * 16777216.0);
  return L;
}

}  // namespace
}  // namespace cwl
