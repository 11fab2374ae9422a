// cwl_stream_*: decode-time scheduler.  One new token per sequence and step (Sec. III-A: complexity is
// estimated as tokens stream in; Sec. III-B: tokens are grouped as they arrive; Sec. III-F: the scheduler keeps its
// state from step to step).
//
// State per sequence, struct of arrays on the device so that thread n's accesses coalesce with its
// neighbours': tokens seen, length and rung of the open chunk, rung of the chunk before it, top-rung
// chunks opened so far, whether the open chunk is the sequence's first, and the quantised (Q24) scores of
// the last min_len tokens (slot = position mod min_len).  One thread advances one sequence:
//   1. the new score enters the trailing window (the last min(min_len, tokens seen) scores);
//   2. the first token opens the first chunk on the window's rung;
//   3. otherwise a chunk of at least min_len tokens is closed when it holds max_len tokens or when the
//      window's rung differs from the rung it was opened on; the token then opens a chunk on the window's
//      rung (one rung lower if that is the top rung and the sequence has used its budget of those);
//   4. the token's row descriptor is written: ranks and scales of its chunk and of the chunk before it and
//      the cross-fade weight lambda = (j+1)/(w+1) for rows j < w of a chunk that is not the first (Sec. III-D).
// All decisions are integer compares of Q24 sums, so the result depends on the fp32 scores only.
#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int kStreamThreads = 128;
constexpr int kStateWords = 6;      // pos, len, cur_rung, prev_rung, hi_used, first

struct StreamLadder {
  int32_t n_rungs, min_len, max_len, window, hi_budget;
  int64_t theta_q[CWL_MAX_RUNGS - 1];  // floor(threshold * 2^24)
  int32_t rung_rank[CWL_MAX_RUNGS];
  float rung_scale[CWL_MAX_RUNGS];
};

__device__ __forceinline__ int32_t stream_quantise(float s) {
  if (s != s) return kQ24;  // NaN: hardest
  s = fminf(fmaxf(s, 0.f), 1.f);
  return __float2int_rd(s * 16777216.0f);  // exact: power-of-two scaling, then floor
}

__device__ __forceinline__ int stream_rung(int64_t sum, int64_t len, const StreamLadder& L) {
  int k = 0;
#pragma unroll
  for (int j = 0; j < CWL_MAX_RUNGS - 1; ++j)
    if (j + 1 < L.n_rungs && sum >= L.theta_q[j] * len) ++k;
  return k;
}

__global__ void __launch_bounds__(kStreamThreads)
stream_reset_kernel(int32_t* words, int n_words) {
  const int i = blockIdx.x * kStreamThreads + threadIdx.x;
  if (i < n_words) words[i] = 0;
}

__global__ void __launch_bounds__(kStreamThreads)
stream_step_kernel(const float* __restrict__ score, const int32_t* __restrict__ active, int n_seq,
                   const __grid_constant__ StreamLadder L, int32_t* __restrict__ state, int32_t* __restrict__ ring,
                   cwl_row_gate* __restrict__ gates) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = blockIdx.x * kStreamThreads + threadIdx.x;
  if (n >= n_seq) return;
  cwl_row_gate g;
  g.rank_in = 0; g.rank_out = 0; g.scale_in = 0.f; g.scale_out = 0.f; g.lambda = 1.f; g.pos_in_chunk = -1; g.opened = 0;
  if (active != nullptr && active[n] == 0) { gates[n] = g; return; }    // sequence not stepping: state untouched

  int32_t* pos_p = state + 0 * n_seq + n;
  int32_t* len_p = state + 1 * n_seq + n;
  int32_t* cur_p = state + 2 * n_seq + n;
  int32_t* prev_p = state + 3 * n_seq + n;
  int32_t* hi_p = state + 4 * n_seq + n;
  int32_t* first_p = state + 5 * n_seq + n;
  const int pos = *pos_p;
  int len = *len_p, cur = *cur_p, prev = *prev_p, hi_used = *hi_p, first = *first_p;

  // 1. trailing window: slots 0 .. n_win-1 hold exactly the last n_win scores
  ring[(int64_t)(pos % L.min_len) * n_seq + n] = stream_quantise(score[n]);
  const int n_win = min(pos + 1, L.min_len);
  int64_t win = 0;
  for (int i = 0; i < n_win; ++i) win += ring[(int64_t)i * n_seq + n];
  int r_win = stream_rung(win, n_win, L);

  // 2./3. does this token open a chunk?
  bool open = false;
  if (pos == 0) { open = true; first = 1; }
  else if (len >= L.min_len && (len >= L.max_len || r_win != cur)) { open = true; first = 0; }
  if (open) {
    if (L.hi_budget >= 0 && L.n_rungs >= 2 && r_win == L.n_rungs - 1) {
      if (hi_used >= L.hi_budget) r_win = L.n_rungs - 2; else hi_used += 1;
    }
    prev = (pos == 0) ? -1 : cur;
    cur = r_win;
    len = 0;
  }

  // 4. the row descriptor of this token
  const int j = len;
  g.pos_in_chunk = j;
  g.opened = open ? 1 : 0;
  g.rank_in = L.rung_rank[cur];
  g.scale_in = L.rung_scale[cur];
  if (!first && j < L.window) {
    g.lambda = __fdiv_rn((float)(j + 1), (float)(L.window + 1));
    g.rank_out = L.rung_rank[prev];
    g.scale_out = L.rung_scale[prev];
  }
  gates[n] = g;
  *pos_p = pos + 1; *len_p = len + 1; *cur_p = cur; *prev_p = prev; *hi_p = hi_used; *first_p = first;
}

bool stream_policy_ok(const cwl_policy* p) {
  if (p == nullptr || p->n_rungs < 1 || p->n_rungs > CWL_MAX_RUNGS) return false;
  if (p->min_len < 1 || p->max_len < p->min_len || p->min_len > CWL_STREAM_MAX_MIN_LEN) return false;
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

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_stream_state_bytes(int32_t n_seq, int32_t min_len) {
  if (n_seq < 0 || min_len < 1 || min_len > CWL_STREAM_MAX_MIN_LEN) return 0;
  return sizeof(int32_t) * (size_t)n_seq * (size_t)(cwl::kStateWords + min_len);
}

extern "C" cwl_status cwl_stream_reset(void* state, size_t state_bytes, int32_t n_seq, int32_t min_len, void* stream) {
  if (n_seq < 0 || min_len < 1 || min_len > CWL_STREAM_MAX_MIN_LEN) return CWL_ERR_INVALID_ARG;
  if (n_seq == 0) return CWL_OK;
  const size_t need = cwl_stream_state_bytes(n_seq, min_len);
  if (state == nullptr || state_bytes < need || (reinterpret_cast<uintptr_t>(state) & 15u) != 0) return CWL_ERR_WORKSPACE;
  const int n_words = (int)(need / sizeof(int32_t));
  cwl::stream_reset_kernel<<<cwl::ceil_div(n_words, cwl::kStreamThreads), cwl::kStreamThreads, 0,
                             static_cast<cudaStream_t>(stream)>>>(static_cast<int32_t*>(state), n_words);
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
}

extern "C" cwl_status cwl_stream_step(const float* score, const int32_t* active, int32_t n_seq,
                                      const cwl_policy* policy, void* state, size_t state_bytes,
                                      cwl_row_gate* gates, void* stream) {
  if (n_seq < 0 || !cwl::stream_policy_ok(policy)) return CWL_ERR_INVALID_ARG;
  if (n_seq == 0) return CWL_OK;
  if (score == nullptr || gates == nullptr) return CWL_ERR_INVALID_ARG;
  const size_t need = cwl_stream_state_bytes(n_seq, policy->min_len);
  if (state == nullptr || state_bytes < need || (reinterpret_cast<uintptr_t>(state) & 15u) != 0) return CWL_ERR_WORKSPACE;
  cwl::StreamLadder L;
  L.n_rungs = policy->n_rungs; L.min_len = policy->min_len; L.max_len = policy->max_len;
  L.window = policy->window; L.hi_budget = policy->hi_budget;
  for (int k = 0; k < CWL_MAX_RUNGS; ++k) {
    L.rung_rank[k] = k < policy->n_rungs ? policy->rung_rank[k] : 0;
    L.rung_scale[k] = k < policy->n_rungs ? policy->rung_scale[k] : 0.f;
  }
  for (int k = 0; k < CWL_MAX_RUNGS - 1; ++k)
    L.theta_q[k] = k + 1 < policy->n_rungs ? (int64_t)__builtin_floor((double)policy->threshold[k] * 16777216.0) : 0;
  int32_t* words = static_cast<int32_t*>(state);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CWL_CUDA_TRY(cwl::launch_chained(!cwl::stream_is_capturing(st), cwl::stream_step_kernel,
                                   dim3(cwl::ceil_div(n_seq, cwl::kStreamThreads)), dim3(cwl::kStreamThreads), 0, st, score,
                                   active, n_seq, L, words, words + (size_t)cwl::kStateWords * n_seq, gates));
  return CWL_OK;
}
