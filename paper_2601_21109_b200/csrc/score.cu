// cwl_score_tokens: token complexity estimator, entropy signal (Sec. III-A (i), Sec. IV-A).
//
// One pass over logits[T, V] (HBM-bound: 4 V bytes per token, one fp32 out).  Each block owns a
// row; every thread keeps an online triple (m, S, U) with
//     m = running max,  S = sum 2^(t),  U = sum t 2^(t),  t = (z - m) log2(e)
// and rescales it when a larger max shows up, so the row is read exactly once.  Triples are
// merged with warp shuffles, then across warps through shared memory.
#include <math_constants.h>

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreBatch = 4;        // 16-byte loads in flight per thread
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct Triple {
  float m, S, U;  // U is kept in the log2 domain: sum t * 2^t
};

// Moves a triple to a new (not smaller) max.  m == -inf means "nothing seen yet".
__device__ __forceinline__ void rebase(Triple& a, float m_new) {
  float dt = (a.m - m_new) * kLog2e;      // <= 0, -inf for an empty triple
  float sc = ex2_approx(dt);
  a.U = (sc > 0.f) ? (a.U + dt * a.S) * sc : 0.f;
  a.S = (sc > 0.f) ? a.S * sc : 0.f;
  a.m = m_new;
}

__device__ __forceinline__ void absorb(Triple& a, float z, float m) {
  // z - m first (exact when z == m, even for huge |m|), then into the log2 domain
  float t = fmaxf((z - m) * kLog2e, -1.0e30f);  // z = -inf: weight 0 and product 0 instead of NaN
  float e = ex2_approx(t);
  a.S += e;
  a.U = fmaf(t, e, a.U);
}

__device__ __forceinline__ Triple merge(Triple a, Triple b) {
  float m = fmaxf(a.m, b.m);
  if (m == -CUDART_INF_F) return a;       // both empty
  rebase(a, m);
  rebase(b, m);
  a.S += b.S;
  a.U += b.U;
  return a;
}

// Further signals of Sec. III-A mixed into the score (kMixed): (ii) n-gram novelty against the previous
// `context` positions of the same sequence, (iv) a positional prior max(0, 1 - p / prior_span).
struct MixParams {
  const int32_t* token_ids;   // [T]
  const int32_t* cu_seqlens;  // [n_seq + 1]
  int n_seq;
  float w_entropy, w_novelty, w_prior;
  int ngram, context, prior_span;
};

template <bool kMixed>
__global__ void __launch_bounds__(kScoreThreads)
score_rows_kernel(const float* __restrict__ logits, int64_t ld, int T, int V, float* __restrict__ score,
                  const MixParams mp) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ Triple warp_part[kScoreThreads / 32];
  __shared__ int warp_bad[kScoreThreads / 32];
  __shared__ int seq_start;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float inv_ln_v = 1.0f / logf((float)V);

  for (int row = blockIdx.x; row < T; row += gridDim.x) {
    const float* z = logits + (int64_t)row * ld;
    int novel = 1, p_in_seq = 0;
    if (kMixed) {
      // the row's sequence (binary search by one thread), then every thread compares the n-gram ending at this
      // token with the n-grams ending at its share of the previous `context` positions
      if (tid == 0) {
        int lo = 0, hi = mp.n_seq;                   // cu[lo] <= row < cu[hi]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (mp.cu_seqlens[mid] <= row) lo = mid; else hi = mid;
        }
        seq_start = mp.cu_seqlens[lo];
      }
      __syncthreads();
      const int start = seq_start;
      p_in_seq = row - start;
      int found = 0;
      if (p_in_seq >= mp.ngram - 1) {
        const int lo = max(row - mp.context, start + mp.ngram - 1);
        for (int u = row - 1 - tid; u >= lo; u -= kScoreThreads) {
          bool same = true;
          for (int i = 0; i < mp.ngram; ++i) same = same && (mp.token_ids[u - i] == mp.token_ids[row - i]);
          found |= same ? 1 : 0;
        }
      }
      novel = __syncthreads_or(found) ? 0 : 1;
    }
    Triple acc{-CUDART_INF_F, 0.f, 0.f};
    bool ok = true;  // stays true while every logit is finite or -inf

    // scalar head up to the first 16-byte boundary, vector body, scalar tail
    int head = (int)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(z) & 15u)) & 15u) >> 2);
    head = min(head, V);
    const int n_vec = (V - head) >> 2;
    const int tail_start = head + (n_vec << 2);

    auto take_scalar = [&](float v) {
      ok = ok && (v < CUDART_INF_F);
      float m_new = fmaxf(acc.m, v);
      if (m_new == -CUDART_INF_F) return;
      if (m_new > acc.m) rebase(acc, m_new);
      absorb(acc, v, acc.m);
    };
    if (tid < head) take_scalar(z[tid]);
    if (tid < V - tail_start) take_scalar(z[tail_start + tid]);

    const float4* zv = reinterpret_cast<const float4*>(z + head);
    // kScoreBatch 16-byte loads are in flight per thread before the first of them is used (a loop that loads and
    // absorbs element by element leaves the compiler one or two loads ahead: 4.7 TB/s against 5.5 TB/s on 2048 rows)
    for (int i = tid; i < n_vec; i += kScoreThreads * kScoreBatch) {
      float4 vv[kScoreBatch];
#pragma unroll
      for (int u = 0; u < kScoreBatch; ++u) {
        const int idx = i + u * kScoreThreads;
        vv[u] = idx < n_vec ? __ldg(zv + idx) : make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
      }
#pragma unroll
      for (int u = 0; u < kScoreBatch; ++u) {
        const float4 v = vv[u];                 // a padding entry (-inf) contributes nothing, like any -inf logit
        ok = ok && (v.x < CUDART_INF_F) && (v.y < CUDART_INF_F) && (v.z < CUDART_INF_F) && (v.w < CUDART_INF_F);
        float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
        float m_new = fmaxf(acc.m, m4);
        if (m_new == -CUDART_INF_F) continue;
        if (m_new > acc.m) rebase(acc, m_new);
        const float m = acc.m;
        absorb(acc, v.x, m);
        absorb(acc, v.y, m);
        absorb(acc, v.z, m);
        absorb(acc, v.w, m);
      }
    }

    int bad = ok ? 0 : 1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Triple o;
      o.m = __shfl_xor_sync(0xffffffffu, acc.m, off);
      o.S = __shfl_xor_sync(0xffffffffu, acc.S, off);
      o.U = __shfl_xor_sync(0xffffffffu, acc.U, off);
      bad |= __shfl_xor_sync(0xffffffffu, bad, off);
      acc = merge(acc, o);
    }
    if (lane == 0) { warp_part[wid] = acc; warp_bad[wid] = bad; }
    __syncthreads();
    if (wid == 0) {
      Triple a = (lane < kScoreThreads / 32) ? warp_part[lane] : Triple{-CUDART_INF_F, 0.f, 0.f};
      int b = (lane < kScoreThreads / 32) ? warp_bad[lane] : 0;
#pragma unroll
      for (int off = 4; off > 0; off >>= 1) {
        Triple o;
        o.m = __shfl_xor_sync(0xffffffffu, a.m, off);
        o.S = __shfl_xor_sync(0xffffffffu, a.S, off);
        o.U = __shfl_xor_sync(0xffffffffu, a.U, off);
        b |= __shfl_xor_sync(0xffffffffu, b, off);
        a = merge(a, o);
      }
      if (lane == 0) {
        float s;
        if (b || a.m == -CUDART_INF_F) {
          s = CUDART_NAN_F;               // NaN / +inf logit, or a row of -inf only
        } else {
          // H = ln S - (U ln2) / S  with U in the log2 domain
          float H = logf(a.S) - (a.U * kLn2) / a.S;
          s = fminf(fmaxf(H * inv_ln_v, 0.f), 1.f);
          if (kMixed) {
            const float prior = fmaxf(0.f, 1.f - (float)p_in_seq / (float)mp.prior_span);
            const float v = mp.w_entropy * s + mp.w_novelty * (float)novel + mp.w_prior * prior;
            s = fminf(fmaxf(v, 0.f), 1.f);
          }
        }
        score[row] = s;
      }
    }
    __syncthreads();
  }
}

}  // namespace
}  // namespace cwl

extern "C" cwl_status cwl_score_tokens(const float* logits, int64_t ld_logits, int32_t T, int32_t V,
                                       float* score, void* stream) {
  if (T < 0 || V < 2) return CWL_ERR_INVALID_ARG;
  if (T == 0) return CWL_OK;
  if (logits == nullptr || score == nullptr) return CWL_ERR_INVALID_ARG;
  if (ld_logits < V) return CWL_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(logits) & 3u) != 0) return CWL_ERR_SHAPE;
  int grid = T < (1 << 20) ? T : (1 << 20);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CWL_CUDA_TRY(cwl::launch_chained(!cwl::stream_is_capturing(st), cwl::score_rows_kernel<false>, dim3(grid),
                                   dim3(cwl::kScoreThreads), 0, st, logits, ld_logits, T, V, score, cwl::MixParams{}));
  return CWL_OK;
}

extern "C" cwl_status cwl_score_tokens_mixed(const float* logits, int64_t ld_logits, int32_t T, int32_t V,
                                             const int32_t* token_ids, const int32_t* cu_seqlens, int32_t n_seq,
                                             const cwl_signal_mix* mix, float* score, void* stream) {
  if (T < 0 || V < 2 || n_seq < 0 || mix == nullptr) return CWL_ERR_INVALID_ARG;
  if (mix->ngram < 1 || mix->ngram > 8 || mix->context < 1 || mix->prior_span < 1) return CWL_ERR_INVALID_ARG;
  if (!(mix->w_entropy >= 0.f) || !(mix->w_novelty >= 0.f) || !(mix->w_prior >= 0.f)) return CWL_ERR_INVALID_ARG;
  if (T == 0) return CWL_OK;
  if (logits == nullptr || score == nullptr || token_ids == nullptr || cu_seqlens == nullptr || n_seq < 1)
    return CWL_ERR_INVALID_ARG;
  if (ld_logits < V) return CWL_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(logits) & 3u) != 0) return CWL_ERR_SHAPE;
  cwl::MixParams mp{token_ids, cu_seqlens, n_seq, mix->w_entropy, mix->w_novelty, mix->w_prior,
                    mix->ngram, mix->context, mix->prior_span};
  int grid = T < (1 << 20) ? T : (1 << 20);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CWL_CUDA_TRY(cwl::launch_chained(!cwl::stream_is_capturing(st), cwl::score_rows_kernel<true>, dim3(grid),
                                   dim3(cwl::kScoreThreads), 0, st, logits, ld_logits, T, V, score, mp));
  return CWL_OK;
}
