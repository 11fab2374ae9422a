// cwl_probe_read (test build only): how fast can ONE launch of the apply kernel's shape read a region of HBM?
// 148 CTAs, one per SM, each streams its slice of the region into a shared-memory ring of the size the apply
// kernel uses (192 KB) with contiguous bulk copies, and drops the data: no tensor-core work, no epilogue, no
// hand-over.  Timed back to back over regions larger than L2, this is the ceiling of a decode-sized launch whose
// operands are read exactly once.  Every wait is bounded; a wait that runs out sets CWL_ERR_TIMEOUT and the CTA
// leaves.
#ifdef CWL_TEST_HOOKS
#include "cwl_common.cuh"

namespace cwl {
namespace {

constexpr int kProbePiece = 16 * 1024;
constexpr int kProbeStages = 12;                 // 192 KB in flight per SM
constexpr unsigned long long kProbeWaitNs = 2000000000ull;

__global__ void __launch_bounds__(32, 1)
probe_read_kernel(const unsigned char* __restrict__ ptr, unsigned long long bytes, int32_t* status_word) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ __align__(8) unsigned long long bars[kProbeStages];
  pdl_launch_dependents();
  const unsigned ring_addr = (unsigned)__cvta_generic_to_shared(ring);
  const unsigned bar0 = (unsigned)__cvta_generic_to_shared(bars);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kProbeStages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8u * s));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  pdl_wait();
  if (threadIdx.x != 0) return;
  const unsigned long long n_cta = gridDim.x;
  unsigned long long slice = (bytes / n_cta) & ~(unsigned long long)(kProbePiece - 1);   // whole pieces only
  const unsigned char* src = ptr + (unsigned long long)blockIdx.x * slice;
  const int n_pieces = (int)(slice / kProbePiece);
  bool ok = true;
  for (int i = 0; i < n_pieces + kProbeStages && ok; ++i) {
    const int s = i % kProbeStages;
    if (i >= kProbeStages) {
      // the copy issued kProbeStages pieces ago into this slot must have landed before the slot is reused
      const unsigned parity = ((i / kProbeStages) - 1) & 1u;
      unsigned long long t0 = 0;
      for (unsigned spins = 0;; ++spins) {
        unsigned done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar0 + 8u * s), "r"(parity) : "memory");
        if (done) break;
        if ((spins & 1023u) == 1023u) {
          unsigned long long now;
          asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
          if (t0 == 0) t0 = now;
          else if (now - t0 > kProbeWaitNs) { ok = false; break; }
        }
      }
    }
    if (ok && i < n_pieces) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar0 + 8u * s), "r"(kProbePiece) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(ring_addr + (unsigned)s * kProbePiece), "l"(src + (unsigned long long)i * kProbePiece),
                     "r"(kProbePiece), "r"(bar0 + 8u * s) : "memory");
    }
  }
  if (!ok) flag_status(status_word, CWL_ERR_TIMEOUT);
}

// The same stream with the apply kernel's second source mixed in: for every 16 KB piece from HBM a CTA also copies
// `hot_piece` bytes from a small region that every CTA reads at the same offsets (the rows of X, which sit in L2), into the
// same ring slot.  `n_stages` slots of (16 KB + hot_piece) bytes.
__global__ void __launch_bounds__(32, 1)
probe_mix_kernel(const unsigned char* __restrict__ ptr, unsigned long long bytes, const unsigned char* __restrict__ hot,
                 unsigned long long hot_bytes, unsigned hot_piece, int n_stages, int32_t* status_word) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ __align__(8) unsigned long long bars[kProbeStages];
  pdl_launch_dependents();
  const unsigned ring_addr = (unsigned)__cvta_generic_to_shared(ring);
  const unsigned bar0 = (unsigned)__cvta_generic_to_shared(bars);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kProbeStages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8u * s));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  pdl_wait();
  if (threadIdx.x != 0) return;
  const unsigned long long n_cta = gridDim.x;
  unsigned long long slice = (bytes / n_cta) & ~(unsigned long long)(kProbePiece - 1);   // whole pieces only
  const unsigned char* src = ptr + (unsigned long long)blockIdx.x * slice;
  const int n_pieces = (int)(slice / kProbePiece);
  const unsigned slot = kProbePiece + hot_piece;
  const unsigned n_hot = (unsigned)(hot_bytes / hot_piece);     // >= 1 (checked by the host)
  bool ok = true;
  for (int i = 0; i < n_pieces + n_stages && ok; ++i) {
    const int s = i % n_stages;
    if (i >= n_stages) {
      const unsigned parity = ((i / n_stages) - 1) & 1u;
      unsigned long long t0 = 0;
      for (unsigned spins = 0;; ++spins) {
        unsigned done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar0 + 8u * s), "r"(parity) : "memory");
        if (done) break;
        if ((spins & 1023u) == 1023u) {
          unsigned long long now;
          asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
          if (t0 == 0) t0 = now;
          else if (now - t0 > kProbeWaitNs) { ok = false; break; }
        }
      }
    }
    if (ok && i < n_pieces) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar0 + 8u * s), "r"(slot) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(ring_addr + (unsigned)s * slot), "l"(src + (unsigned long long)i * kProbePiece),
                     "r"(kProbePiece), "r"(bar0 + 8u * s) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(ring_addr + (unsigned)s * slot + kProbePiece), "l"(hot + (unsigned long long)((unsigned)i % n_hot) * hot_piece),
                     "r"(hot_piece), "r"(bar0 + 8u * s) : "memory");
    }
  }
  if (!ok) flag_status(status_word, CWL_ERR_TIMEOUT);
}

}  // namespace
}  // namespace cwl

extern "C" cwl_status cwl_probe_read_mix(const void* ptr, size_t bytes, const void* hot, size_t hot_bytes, uint32_t hot_piece,
                                         int32_t ctas, int32_t* status_word, void* stream_) {
  using namespace cwl;
  if (ptr == nullptr || hot == nullptr || ctas < 1 || ctas > 148 || bytes < (size_t)ctas * kProbePiece ||
      (reinterpret_cast<uintptr_t>(ptr) & 127u) != 0 || (reinterpret_cast<uintptr_t>(hot) & 127u) != 0 ||
      hot_piece < 16 || hot_piece % 16 != 0 || hot_piece > 32 * 1024 || hot_bytes < hot_piece)
    return CWL_ERR_INVALID_ARG;
  const int ring = kProbePiece * kProbeStages;                   // 192 KB
  int n_stages = ring / (int)(kProbePiece + hot_piece);
  if (n_stages > kProbeStages) n_stages = kProbeStages;
  if (n_stages < 2) return CWL_ERR_INVALID_ARG;
  static bool configured = false;
  if (!configured) {
    CWL_CUDA_TRY(cudaFuncSetAttribute(probe_mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ring));
    configured = true;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  CWL_CUDA_TRY(launch_chained(!stream_is_capturing(stream), probe_mix_kernel, dim3(ctas), dim3(32), (size_t)ring, stream,
                              static_cast<const unsigned char*>(ptr), (unsigned long long)bytes,
                              static_cast<const unsigned char*>(hot), (unsigned long long)hot_bytes, (unsigned)hot_piece, n_stages,
                              status_word));
  return CWL_OK;
}

extern "C" cwl_status cwl_probe_read(const void* ptr, size_t bytes, int32_t* status_word, void* stream_) {
  using namespace cwl;
  if (ptr == nullptr || bytes < (size_t)148 * kProbePiece || (reinterpret_cast<uintptr_t>(ptr) & 127u) != 0)
    return CWL_ERR_INVALID_ARG;
  static bool configured = false;
  const int smem = kProbePiece * kProbeStages;
  if (!configured) {
    CWL_CUDA_TRY(cudaFuncSetAttribute(probe_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured = true;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  CWL_CUDA_TRY(launch_chained(!stream_is_capturing(stream), probe_read_kernel, dim3(148), dim3(32), (size_t)smem, stream,
                              static_cast<const unsigned char*>(ptr), (unsigned long long)bytes, status_word));
  return CWL_OK;
}
#endif  // CWL_TEST_HOOKS
