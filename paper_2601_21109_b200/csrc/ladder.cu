// cwl_ladder_build: offline construction of the rank ladder (Sec. III-C: the trained update A B is re-factorised
// once by SVD so that every prefix of the stored factors is a usable adapter).
//
//   A B = U diag(sigma) V^T,  A' = U diag(sigma) [d_in, R],  B' = V^T [R, d_out],  sigma descending,
// so that A'[:, :r] B'[:r, :] is the best rank-r approximation of A B for every r (Eckart-Young).
//
// Two one-sided (Hestenes) Jacobi passes in fp64, never forming the d_in x d_out product or a Gram matrix:
//   1. rotate the columns of B^T (d_out x R) until they are orthogonal:  B^T Vb = Ub Sb;
//   2. C = A Vb Sb (d_in x R), rotate its columns until orthogonal:      C Vc = Uc Sc;
// then A B = C Ub^T = Uc Sc (Ub Vc)^T: A' is the rotated C, B' = Vc^T Ub^T, both re-ordered by descending sigma.
// A Jacobi step rotates R/2 disjoint column pairs (round-robin schedule), one block per pair; R-1 steps make a
// sweep; sweeps repeat until no pair's cosine exceeds 1e-14 (checked on the host once per sweep: this is an
// offline routine and synchronises the stream).
#include <cuda_bf16.h>

#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int kJacThreads = 256;
constexpr int kMaxSweeps = 40;
constexpr double kJacTol = 1e-14;

__device__ __forceinline__ double block_sum(double v, double* scratch) {
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) scratch[wid] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kJacThreads / 32; ++w) t += scratch[w];
  return t;
}

// X [n x R] column-major fp64 <- transpose-free load of a bf16 row-major matrix M [R rows x n cols] (column j of X
// is row j of M), or of M [n rows x R cols] when `rows_are_columns` is false.
__global__ void load_columns_kernel(const __nv_bfloat16* M, int64_t ld, int n, int R, bool rows_are_columns, double* X) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * R) return;
  const int j = (int)(idx / n), i = (int)(idx - (int64_t)j * n);
  X[idx] = rows_are_columns ? (double)__bfloat162float(M[(int64_t)j * ld + i]) : (double)__bfloat162float(M[(int64_t)i * ld + j]);
}

__global__ void identity_kernel(double* V, int R) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < R * R) V[idx] = (idx / R == idx % R) ? 1.0 : 0.0;
}

// One step of a sweep: block k rotates the column pair the round-robin schedule gives it.
__global__ void __launch_bounds__(kJacThreads)
jacobi_step_kernel(double* X, int n, int R, double* V, int step, double* worst) {
  __shared__ double scratch[kJacThreads / 32];
  const int k = blockIdx.x, m = R - 1;
  int p, q;
  if (k == 0) { p = m; q = step; }
  else { p = (step + k) % m; q = (step - k + m) % m; }
  double* xp = X + (int64_t)p * n;
  double* xq = X + (int64_t)q * n;
  double a = 0.0, b = 0.0, g = 0.0;
  for (int i = threadIdx.x; i < n; i += kJacThreads) {
    const double u = xp[i], v = xq[i];
    a += u * u; b += v * v; g += u * v;
  }
  a = block_sum(a, scratch); b = block_sum(b, scratch); g = block_sum(g, scratch);
  const double denom = sqrt(a * b);
  if (denom == 0.0 || fabs(g) <= kJacTol * denom) return;          // already orthogonal (or a zero column)
  if (threadIdx.x == 0) {
    // max over the sweep of the pairs' |cosine|: positive doubles order like their bit patterns
    atomicMax(reinterpret_cast<unsigned long long*>(worst), (unsigned long long)__double_as_longlong(fabs(g) / denom));
  }
  const double zeta = (b - a) / (2.0 * g);
  const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
  const double c = 1.0 / sqrt(1.0 + t * t), s = c * t;
  for (int i = threadIdx.x; i < n; i += kJacThreads) {
    const double u = xp[i], v = xq[i];
    xp[i] = c * u - s * v;
    xq[i] = s * u + c * v;
  }
  double* vp = V + (int64_t)p * R;
  double* vq = V + (int64_t)q * R;
  for (int i = threadIdx.x; i < R; i += kJacThreads) {
    const double u = vp[i], v = vq[i];
    vp[i] = c * u - s * v;
    vq[i] = s * u + c * v;
  }
}

// norm[j] = || X[:, j] ||
__global__ void __launch_bounds__(kJacThreads)
column_norms_kernel(const double* X, int n, double* norm) {
  __shared__ double scratch[kJacThreads / 32];
  const double* x = X + (int64_t)blockIdx.x * n;
  double a = 0.0;
  for (int i = threadIdx.x; i < n; i += kJacThreads) a += x[i] * x[i];
  a = block_sum(a, scratch);
  if (threadIdx.x == 0) norm[blockIdx.x] = sqrt(a);
}

// C[:, i] = (A Vb)[:, i] * sb[i]      (A bf16 [d_in, R] row-major, Vb column-major [R x R], C column-major)
__global__ void project_kernel(const __nv_bfloat16* A, int64_t lda, int d_in, int R, const double* Vb, const double* sb,
                               double* C) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)d_in * R) return;
  const int i = (int)(idx / d_in), m = (int)(idx - (int64_t)i * d_in);
  double acc = 0.0;
  for (int j = 0; j < R; ++j) acc += (double)__bfloat162float(A[(int64_t)m * lda + j]) * Vb[(int64_t)i * R + j];
  C[idx] = acc * sb[i];
}

// place[i] = position of column i when the columns are sorted by descending norm (ties: lower index first)
__global__ void order_kernel(const double* norm, int R, int* place) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= R) return;
  int r = 0;
  for (int j = 0; j < R; ++j) r += (norm[j] > norm[i] || (norm[j] == norm[i] && j < i)) ? 1 : 0;
  place[i] = r;
}

// A'[m, place[i]] = C'[m, i]  (C' = rotated C, column-major), fp32 and / or bf16, row-major [d_in, R]
__global__ void emit_left_kernel(const double* C, int d_in, int R, const int* place, float* A32, int64_t ld32,
                                 __nv_bfloat16* A16, int64_t ld16) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)d_in * R) return;
  const int i = (int)(idx / d_in), m = (int)(idx - (int64_t)i * d_in);
  const double v = C[idx];
  if (A32 != nullptr) A32[(int64_t)m * ld32 + place[i]] = (float)v;
  if (A16 != nullptr) A16[(int64_t)m * ld16 + place[i]] = __float2bfloat16_rn((float)v);
}

// B'[place[i], n] = sum_j Vc[j, i] Xb'[n, j] / sb[j]   (Ub = Xb' Sb^-1; directions with sb ~ 0 carry nothing)
__global__ void emit_right_kernel(const double* Xb, int d_out, int R, const double* Vc, const double* sb, double sb_floor,
                                  const int* place, float* B32, int64_t ld32, __nv_bfloat16* B16, int64_t ld16) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)d_out * R) return;
  const int i = (int)(idx / d_out), n = (int)(idx - (int64_t)i * d_out);
  double acc = 0.0;
  for (int j = 0; j < R; ++j)
    if (sb[j] > sb_floor) acc += Vc[(int64_t)i * R + j] * Xb[(int64_t)j * d_out + n] / sb[j];
  if (B32 != nullptr) B32[(int64_t)place[i] * ld32 + n] = (float)acc;
  if (B16 != nullptr) B16[(int64_t)place[i] * ld16 + n] = __float2bfloat16_rn((float)acc);
}

__global__ void emit_sigma_kernel(const double* norm, int R, const int* place, float* sigma) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < R) sigma[place[i]] = (float)norm[i];
}

struct LadderWorkspace { double *Xb, *Xc, *Vb, *Vc, *sb, *sc, *worst; int* place; };

size_t carve_ladder(LadderWorkspace& w, char* base, int d_in, int d_out, int R) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  size_t off = 0;
  auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off = up(off + bytes); return p; };
  w.Xb = reinterpret_cast<double*>(take(sizeof(double) * (size_t)d_out * R));
  w.Xc = reinterpret_cast<double*>(take(sizeof(double) * (size_t)d_in * R));
  w.Vb = reinterpret_cast<double*>(take(sizeof(double) * (size_t)R * R));
  w.Vc = reinterpret_cast<double*>(take(sizeof(double) * (size_t)R * R));
  w.sb = reinterpret_cast<double*>(take(sizeof(double) * R));
  w.sc = reinterpret_cast<double*>(take(sizeof(double) * R));
  w.worst = reinterpret_cast<double*>(take(sizeof(double)));
  w.place = reinterpret_cast<int*>(take(sizeof(int) * R));
  return off;
}

// Sweeps until every pair is orthogonal to kJacTol.  Synchronises the stream once per sweep.
cwl_status jacobi(double* X, int n, int R, double* V, double* worst, cudaStream_t stream, int* sweeps_out) {
  identity_kernel<<<ceil_div(R * R, 256), 256, 0, stream>>>(V, R);
  int sweeps = 0;
  for (; sweeps < kMaxSweeps; ++sweeps) {
    CWL_CUDA_TRY(cudaMemsetAsync(worst, 0, sizeof(double), stream));
    for (int step = 0; step < R - 1; ++step)
      jacobi_step_kernel<<<R / 2, kJacThreads, 0, stream>>>(X, n, R, V, step, worst);
    double h = 0.0;
    CWL_CUDA_TRY(cudaMemcpyAsync(&h, worst, sizeof(double), cudaMemcpyDeviceToHost, stream));
    CWL_CUDA_TRY(cudaStreamSynchronize(stream));
    if (h == 0.0) { ++sweeps; break; }             // no pair needed a rotation in this sweep
  }
  if (sweeps_out != nullptr) *sweeps_out += sweeps;
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
}

}  // namespace
}  // namespace cwl

extern "C" size_t cwl_ladder_workspace_bytes(int32_t d_in, int32_t d_out, int32_t R) {
  if (d_in < 1 || d_out < 1 || R < 2) return 0;
  cwl::LadderWorkspace w;
  return cwl::carve_ladder(w, nullptr, d_in, d_out, R);
}

extern "C" cwl_status cwl_ladder_build(const void* A, int64_t lda, const void* B, int64_t ldb,
                                       int32_t d_in, int32_t d_out, int32_t R,
                                       void* A_out, int64_t lda_out, void* B_out, int64_t ldb_out,
                                       float* A_out_f32, float* B_out_f32, float* sigma,
                                       void* workspace, size_t workspace_bytes, int32_t* sweeps, void* stream_) {
  using namespace cwl;
  if (A == nullptr || B == nullptr || d_in < 1 || d_out < 1) return CWL_ERR_INVALID_ARG;
  if (R < 2 || R % 2 != 0 || R > CWL_MAX_RANK || R > d_in || R > d_out) return CWL_ERR_UNSUPPORTED;
  if (lda < R || ldb < d_out || (A_out != nullptr && lda_out < R) || (B_out != nullptr && ldb_out < d_out)) return CWL_ERR_SHAPE;
  LadderWorkspace w;
  const size_t need = carve_ladder(w, static_cast<char*>(workspace), d_in, d_out, R);
  if (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return CWL_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const __nv_bfloat16* Ab = static_cast<const __nv_bfloat16*>(A);
  const __nv_bfloat16* Bb = static_cast<const __nv_bfloat16*>(B);
  if (sweeps != nullptr) *sweeps = 0;

  // 1. B^T Vb = Ub Sb
  load_columns_kernel<<<(int)ceil_div64((int64_t)d_out * R, 256), 256, 0, stream>>>(Bb, ldb, d_out, R, true, w.Xb);
  cwl_status st = jacobi(w.Xb, d_out, R, w.Vb, w.worst, stream, sweeps);
  if (st != CWL_OK) return st;
  column_norms_kernel<<<R, kJacThreads, 0, stream>>>(w.Xb, d_out, w.sb);
  // 2. C = A Vb Sb,  C Vc = Uc Sc
  project_kernel<<<(int)ceil_div64((int64_t)d_in * R, 256), 256, 0, stream>>>(Ab, lda, d_in, R, w.Vb, w.sb, w.Xc);
  st = jacobi(w.Xc, d_in, R, w.Vc, w.worst, stream, sweeps);
  if (st != CWL_OK) return st;
  column_norms_kernel<<<R, kJacThreads, 0, stream>>>(w.Xc, d_in, w.sc);
  order_kernel<<<ceil_div(R, 256), 256, 0, stream>>>(w.sc, R, w.place);
  // 3. outputs.  Directions of B below 1e-13 of its largest are treated as absent.
  double sb_host[CWL_MAX_RANK];
  CWL_CUDA_TRY(cudaMemcpyAsync(sb_host, w.sb, sizeof(double) * R, cudaMemcpyDeviceToHost, stream));
  CWL_CUDA_TRY(cudaStreamSynchronize(stream));
  double sb_max = 0.0;
  for (int j = 0; j < R; ++j) if (sb_host[j] > sb_max) sb_max = sb_host[j];
  emit_left_kernel<<<(int)ceil_div64((int64_t)d_in * R, 256), 256, 0, stream>>>(
      w.Xc, d_in, R, w.place, A_out_f32, R, static_cast<__nv_bfloat16*>(A_out), lda_out);
  emit_right_kernel<<<(int)ceil_div64((int64_t)d_out * R, 256), 256, 0, stream>>>(
      w.Xb, d_out, R, w.Vc, w.sb, sb_max * 1e-13, w.place, B_out_f32, d_out, static_cast<__nv_bfloat16*>(B_out), ldb_out);
  if (sigma != nullptr) emit_sigma_kernel<<<ceil_div(R, 256), 256, 0, stream>>>(w.sc, R, w.place, sigma);
  CWL_CUDA_TRY(cudaGetLastError());
  return CWL_OK;
}
