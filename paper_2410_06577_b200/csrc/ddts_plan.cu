// Varlen bookkeeping on the device: checks cu_seqlens, resets the workspace header and writes
// the order in which persistent CTAs should take sequences (longest first, so that the last
// CTAs to finish hold short sequences).  One small CTA; runs before the prefill kernel on the
// same stream.
#include "ddts_common.cuh"

namespace ddts {
namespace {

constexpr int kPlanThreads = 1024;

__global__ void __launch_bounds__(kPlanThreads, 1)
ddts_plan_kernel(const int32_t* __restrict__ cu, int N, int T, WorkspaceHeader* hdr,
                 int32_t* __restrict__ order) {
  __shared__ int s_bad;
  __shared__ int s_len[kMaxSortedSeqs];
  const int tid = threadIdx.x;
  if (tid == 0) s_bad = 0;
  __syncthreads();
  int bad = 0;
  for (int n = tid; n < N; n += kPlanThreads) {
    const int lo = cu[n], hi = cu[n + 1];
    if (hi < lo || lo < 0 || hi > T) bad = 1;
    if (n < kMaxSortedSeqs) {
      const int clo = lo < 0 ? 0 : (lo > T ? T : lo);
      const int chi = hi < clo ? clo : (hi > T ? T : hi);
      s_len[n] = chi - clo;
    }
  }
  if (tid == 0 && (cu[0] != 0 || cu[N] != T)) bad = 1;
  if (bad) atomicOr(&s_bad, 1);
  __syncthreads();
  if (tid == 0) {
    hdr->status = s_bad ? (int)RODIMUS_ERR_SEQLENS : (int)RODIMUS_OK;
  }
  const int ns = N < kMaxSortedSeqs ? N : kMaxSortedSeqs;
  for (int n = tid; n < N; n += kPlanThreads) {
    if (n >= ns) {
      order[n] = n;
      continue;
    }
    const int len = s_len[n];
    int rank = 0;
    for (int j = 0; j < ns; ++j) {
      const int lj = s_len[j];
      rank += (lj > len) || (lj == len && j < n);
    }
    order[rank] = n;
  }
}

}  // namespace

cudaError_t launch_plan(const rodimus_ddts_fwd_params& p, int* n_launches) {
  *n_launches = 0;
  auto* hdr = reinterpret_cast<WorkspaceHeader*>(p.workspace);
  auto* order = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(p.workspace) + sizeof(WorkspaceHeader));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(p.stream);
  ddts_plan_kernel<<<1, kPlanThreads, 0, st>>>(p.cu_seqlens, p.N, p.T, hdr, order);
  *n_launches = 1;
  return cudaGetLastError();
}

}  // namespace ddts
