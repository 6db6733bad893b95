// Host side of the C ABI: argument checks (before any launch), workspace sizing, kernel choice.
#include <cstring>

#include "ddts_common.cuh"

namespace {

thread_local int t_last_launches = 0;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t workspace_bytes_for(int n_seq) {
  size_t order = (size_t)(n_seq > 0 ? n_seq : 0) * sizeof(int32_t);
  order = (order + 255) & ~(size_t)255;
  return sizeof(ddts::WorkspaceHeader) + order;
}

// Everything about the sizes that does not need a pointer.
int check_fwd_sizes(const rodimus_ddts_fwd_params* p, bool varlen) {
  if (p->struct_size != (int32_t)sizeof(rodimus_ddts_fwd_params)) return RODIMUS_ERR_DTYPE;
  if (p->dtype != RODIMUS_BF16 && p->dtype != RODIMUS_F32) return RODIMUS_ERR_DTYPE;
  if (p->ingate != RODIMUS_INGATE_POW_G && p->ingate != RODIMUS_INGATE_POW_SIGMOID)
    return RODIMUS_ERR_DTYPE;
  if ((p->shared_gates != 0 && p->shared_gates != 1) || p->reserved != 0) return RODIMUS_ERR_DTYPE;
  if (p->B < 0 || p->H < 0 || p->T < 0) return RODIMUS_ERR_SHAPE;
  if (p->dk <= 0 || p->dv <= 0) return RODIMUS_ERR_SHAPE;
  // well-formed widths that none of the kernels covers
  if (p->dk % 16 || p->dv % 16 || p->dk > 256 || p->dv > 1024) return RODIMUS_ERR_UNSUPPORTED;
  if ((long long)p->B * p->H * p->T >= (1LL << 31)) return RODIMUS_ERR_SHAPE;
  if (varlen) {
    if (p->B != 1 || p->N < 0) return RODIMUS_ERR_SHAPE;
    if ((long long)p->N * p->H >= (1LL << 31)) return RODIMUS_ERR_SHAPE;
  }
  return RODIMUS_OK;
}

}  // namespace

namespace {
constexpr long long kDefaultWaitCycles = 4000000000LL;   // about two seconds
std::atomic<long long> g_wait_cycles{kDefaultWaitCycles};
}  // namespace

namespace ddts {

long long main_loop_wait_cycles() { return g_wait_cycles.load(std::memory_order_relaxed); }

cudaError_t current_device(int* dev, int* sms) {
  static std::atomic<int> cached[64];   // SM count per device ordinal, 0 = not asked yet
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return e;
  const bool slot = *dev >= 0 && *dev < 64;
  int n = slot ? cached[*dev].load(std::memory_order_relaxed) : 0;
  if (n == 0) {
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, *dev);
    if (e != cudaSuccess) return e;
    if (slot) cached[*dev].store(n, std::memory_order_relaxed);
  }
  *sms = n;
  return cudaSuccess;
}

bool fwd_tc_supported(const rodimus_ddts_fwd_params& p) {
  return p.dtype == RODIMUS_BF16 && p.dk == 128 && p.dv % 128 == 0;
}

// the value-side decay (the paper's ablation arm) exists in the fp32 kernel only
bool fwd_pair_selected(const rodimus_ddts_fwd_params& p) { return fwd_pair_supported(p) && !p.value_decay; }

bool has_block_terms(const rodimus_ddts_fwd_params& p) { return p.beta_hat || p.feed_d; }

// 0: cluster-pair tensor-core kernel, 1: single-CTA tensor-core kernel (the recurrence alone),
// 2: fp32 CUDA-core kernel
int fwd_kernel_choice(const rodimus_ddts_fwd_params& p) {
  if (fwd_pair_selected(p)) return 0;
  if (fwd_tc_supported(p) && !has_block_terms(p) && !p.shared_gates && !p.value_decay) return 1;
  return 2;
}

}  // namespace ddts

extern "C" {

size_t rodimus_ddts_fwd_workspace_bytes(const rodimus_ddts_fwd_params* p) {
  if (!p) return 0;
  const bool varlen = p->cu_seqlens != nullptr || p->cu_seqlens_host != nullptr;
  if (check_fwd_sizes(p, varlen) != RODIMUS_OK) return 0;
  const size_t base = workspace_bytes_for(varlen ? p->N : 0);
  // long dense sequences with few heads run faster split along time, given room for the
  // segments' states; a caller that passes only the base size still gets the unsplit path
  const size_t split = ddts::fwd_pair_selected(*p) ? ddts::fwd_pair_split_workspace_bytes(*p) : 0;
  return split > base ? split : base;
}

const char* rodimus_ddts_fwd_kernel_name(const rodimus_ddts_fwd_params* p) {
  if (!p) return "invalid";
  if (check_fwd_sizes(p, p->cu_seqlens != nullptr) != RODIMUS_OK) return "invalid";
  return ddts::fwd_kernel_choice(*p) < 2 ? "tcgen05" : "simt";
}

int rodimus_ddts_fwd(const rodimus_ddts_fwd_params* p) {
  t_last_launches = 0;
  if (!p) return RODIMUS_ERR_NULL;
  const bool varlen = p->cu_seqlens != nullptr;
  int rc = check_fwd_sizes(p, varlen);
  if (rc != RODIMUS_OK) return rc;
  if (!varlen && p->cu_seqlens_host) return RODIMUS_ERR_NULL;  // host copy without the device array
  const long long rows = (long long)p->B * p->H * p->T;
  const long long n_seq = varlen ? p->N : p->B;
  if (rows > 0 && (!p->q || !p->k || !p->gate_x || !p->temp_y || !p->v || !p->o))
    return RODIMUS_ERR_NULL;
  if ((p->feed_d != nullptr) != (p->feed_x != nullptr)) return RODIMUS_ERR_NULL;  // both or neither
  const void* ptrs[] = {p->q, p->k, p->gate_x, p->temp_y, p->v, p->o, p->s0, p->sT, p->cu_seqlens,
                        p->beta_hat, p->feed_d, p->feed_x, p->value_decay};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return RODIMUS_ERR_ALIGN;
  if (!p->workspace || p->workspace_bytes < workspace_bytes_for(varlen ? p->N : 0))
    return RODIMUS_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(p->workspace) & 255u) return RODIMUS_ERR_ALIGN;
  if (varlen && p->cu_seqlens_host) {
    const int32_t* cu = p->cu_seqlens_host;
    if (cu[0] != 0 || cu[p->N] != p->T) return RODIMUS_ERR_SEQLENS;
    for (int n = 0; n < p->N; ++n)
      if (cu[n + 1] < cu[n]) return RODIMUS_ERR_SEQLENS;
  }
  if (varlen && p->N == 0 && p->T != 0) return RODIMUS_ERR_SEQLENS;
  if (n_seq * p->H == 0) return RODIMUS_OK;  // nothing to compute, nothing to write

  int launches = 0, n = 0;
  cudaError_t e = cudaSuccess;
  if (varlen) {  // checks cu_seqlens on the device, clears the status word, orders the work
    e = ddts::launch_plan(*p, &n);
    launches += n;
  }  // dense: the prefill kernel's first CTA clears the status word itself
  if (e != cudaSuccess) return RODIMUS_ERR_CUDA;
  const int choice = ddts::fwd_kernel_choice(*p);
  if (choice == 0)
    e = ddts::launch_fwd_pair(*p, &n);
  else if (choice == 1)
    e = ddts::launch_fwd_tc(*p, &n);
  else
    e = ddts::launch_fwd_simt(*p, &n);
  launches += n;
  if (e != cudaSuccess) return RODIMUS_ERR_CUDA;
  t_last_launches = launches;
  return RODIMUS_OK;
}

static int check_bwd_sizes(const rodimus_ddts_bwd_params* p, bool varlen) {
  if (p->struct_size != (int32_t)sizeof(rodimus_ddts_bwd_params)) return RODIMUS_ERR_DTYPE;
  if (p->dtype != RODIMUS_BF16 && p->dtype != RODIMUS_F32) return RODIMUS_ERR_DTYPE;
  if (p->ingate != RODIMUS_INGATE_POW_G && p->ingate != RODIMUS_INGATE_POW_SIGMOID)
    return RODIMUS_ERR_DTYPE;
  if (p->B < 0 || p->H < 0 || p->T < 0) return RODIMUS_ERR_SHAPE;
  if (p->dk <= 0 || p->dv <= 0) return RODIMUS_ERR_SHAPE;
  if (!ddts::bwd_supported(*p)) return RODIMUS_ERR_UNSUPPORTED;
  if ((long long)p->B * p->H * p->T >= (1LL << 31)) return RODIMUS_ERR_SHAPE;
  if (varlen) {
    if (p->B != 1 || p->N < 0) return RODIMUS_ERR_SHAPE;
    if ((long long)p->N * p->H >= (1LL << 31) / 8) return RODIMUS_ERR_SHAPE;
  }
  return RODIMUS_OK;
}

size_t rodimus_ddts_bwd_workspace_bytes(const rodimus_ddts_bwd_params* p) {
  if (!p) return 0;
  const bool varlen = p->cu_seqlens != nullptr || p->cu_seqlens_host != nullptr;
  if (check_bwd_sizes(p, varlen) != RODIMUS_OK) return 0;
  rodimus_ddts_bwd_params c = *p;
  if (varlen && !c.cu_seqlens) c.cu_seqlens = c.cu_seqlens_host;   // only tested against NULL
  return workspace_bytes_for(varlen ? p->N : 0) + ddts::bwd_scratch_bytes(c);
}

int rodimus_ddts_bwd(const rodimus_ddts_bwd_params* p) {
  t_last_launches = 0;
  if (!p) return RODIMUS_ERR_NULL;
  const bool varlen = p->cu_seqlens != nullptr;
  int rc = check_bwd_sizes(p, varlen);
  if (rc != RODIMUS_OK) return rc;
  if (!varlen && p->cu_seqlens_host) return RODIMUS_ERR_NULL;
  const long long rows = (long long)p->B * p->H * p->T;
  const long long n_seq = varlen ? p->N : p->B;
  if (rows > 0 && (!p->q || !p->k || !p->gate_x || !p->temp_y || !p->v || !p->d_o || !p->d_q ||
                   !p->d_k || !p->d_gate_x || !p->d_temp_y || !p->d_v))
    return RODIMUS_ERR_NULL;
  const void* ptrs[] = {p->q, p->k, p->gate_x, p->temp_y, p->v, p->d_o, p->s0, p->d_sT, p->d_q,
                        p->d_k, p->d_gate_x, p->d_temp_y, p->d_v, p->d_s0, p->cu_seqlens};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return RODIMUS_ERR_ALIGN;
  const size_t base = workspace_bytes_for(varlen ? p->N : 0);
  if (!p->workspace || p->workspace_bytes < base + ddts::bwd_scratch_bytes(*p))
    return RODIMUS_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(p->workspace) & 255u) return RODIMUS_ERR_ALIGN;
  if (varlen && p->cu_seqlens_host) {
    const int32_t* cu = p->cu_seqlens_host;
    if (cu[0] != 0 || cu[p->N] != p->T) return RODIMUS_ERR_SEQLENS;
    for (int n = 0; n < p->N; ++n)
      if (cu[n + 1] < cu[n]) return RODIMUS_ERR_SEQLENS;
  }
  if (varlen && p->N == 0 && p->T != 0) return RODIMUS_ERR_SEQLENS;
  if (n_seq * p->H == 0) return RODIMUS_OK;
  int launches = 0, n = 0;
  cudaError_t e = cudaSuccess;
  if (varlen) {   // device-side check of cu_seqlens into the status word
    rodimus_ddts_fwd_params f;
    std::memset(&f, 0, sizeof(f));
    f.cu_seqlens = p->cu_seqlens; f.N = p->N; f.T = p->T;
    f.workspace = p->workspace; f.stream = p->stream;
    e = ddts::launch_plan(f, &n);
    launches += n;
    if (e != cudaSuccess) return RODIMUS_ERR_CUDA;
  }
  e = ddts::launch_bwd(*p, base, &n);
  launches += n;
  if (e != cudaSuccess) return RODIMUS_ERR_CUDA;
  t_last_launches = launches;
  return RODIMUS_OK;
}

int rodimus_swska_fwd(const rodimus_swska_fwd_params* p) {
  t_last_launches = 0;
  if (!p) return RODIMUS_ERR_NULL;
  if (p->struct_size != (int32_t)sizeof(rodimus_swska_fwd_params)) return RODIMUS_ERR_DTYPE;
  if (p->dtype != RODIMUS_BF16 && p->dtype != RODIMUS_F32) return RODIMUS_ERR_DTYPE;
  if (p->B < 0 || p->H < 0 || p->T < 0 || p->d <= 0 || p->window < 1) return RODIMUS_ERR_SHAPE;
  if (!(p->scale > 0.f) || !(p->scale < 1e30f)) return RODIMUS_ERR_SHAPE;   // positive and finite
  if (!ddts::swska_supported(*p)) return RODIMUS_ERR_UNSUPPORTED;
  if ((long long)p->B * p->H * p->T >= (1LL << 31) || p->B > 65535 || p->H > 65535)
    return RODIMUS_ERR_SHAPE;
  if ((long long)p->B * p->H * p->T == 0) return RODIMUS_OK;
  if (!p->q || !p->k || !p->v || !p->o) return RODIMUS_ERR_NULL;
  const void* ptrs[] = {p->q, p->k, p->v, p->o};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return RODIMUS_ERR_ALIGN;
  if (p->workspace) {
    if (p->workspace_bytes < sizeof(ddts::WorkspaceHeader)) return RODIMUS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(p->workspace) & 255u) return RODIMUS_ERR_ALIGN;
  }
  int n = 0;
  if (ddts::launch_swska(*p, &n) != cudaSuccess) return RODIMUS_ERR_CUDA;
  t_last_launches = n;
  return RODIMUS_OK;
}

int rodimus_ddts_step(const rodimus_ddts_step_params* p) {
  t_last_launches = 0;
  if (!p) return RODIMUS_ERR_NULL;
  if (p->struct_size != (int32_t)sizeof(rodimus_ddts_step_params)) return RODIMUS_ERR_DTYPE;
  if (p->dtype != RODIMUS_BF16 && p->dtype != RODIMUS_F32) return RODIMUS_ERR_DTYPE;
  if (p->ingate != RODIMUS_INGATE_POW_G && p->ingate != RODIMUS_INGATE_POW_SIGMOID)
    return RODIMUS_ERR_DTYPE;
  if ((p->shared_gates != 0 && p->shared_gates != 1) || p->reserved != 0) return RODIMUS_ERR_DTYPE;
  if (p->Nseq < 0 || p->H < 0) return RODIMUS_ERR_SHAPE;
  if (p->dk <= 0 || p->dv <= 0) return RODIMUS_ERR_SHAPE;
  if (p->dk % 16 || p->dv % 16 || p->dk > 256 || p->dv > 1024) return RODIMUS_ERR_UNSUPPORTED;
  if ((long long)p->Nseq * p->H >= (1LL << 31) / 8) return RODIMUS_ERR_SHAPE;
  if ((long long)p->Nseq * p->H == 0) return RODIMUS_OK;
  if (!p->q || !p->k || !p->gate_x || !p->temp_y || !p->v || !p->o || !p->state)
    return RODIMUS_ERR_NULL;
  if ((p->feed_d != nullptr) != (p->feed_x != nullptr)) return RODIMUS_ERR_NULL;
  const void* ptrs[] = {p->q, p->k, p->gate_x, p->temp_y, p->v, p->o, p->state};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return RODIMUS_ERR_ALIGN;
  const void* opt[] = {p->beta_hat, p->feed_d, p->feed_x, p->value_decay};
  for (const void* ptr : opt)
    if (ptr && !aligned16(ptr)) return RODIMUS_ERR_ALIGN;
  int n = 0;
  cudaError_t e = ddts::launch_step(*p, &n);
  if (e != cudaSuccess) return RODIMUS_ERR_CUDA;
  t_last_launches = n;
  return RODIMUS_OK;
}

int rodimus_ddts_device_status(const void* workspace, void* stream) {
  if (!workspace) return RODIMUS_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int32_t status = 0;
  if (cudaMemcpyAsync(&status, workspace, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return RODIMUS_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return RODIMUS_ERR_CUDA;
  return status;
}

int rodimus_ddts_last_launch_count(void) { return t_last_launches; }

int rodimus_ddts_test_set_wait_limit(long long cycles) {
  g_wait_cycles.store(cycles < 0 ? kDefaultWaitCycles : cycles, std::memory_order_relaxed);
  return RODIMUS_OK;
}

const char* rodimus_status_str(int status) {
  switch (status) {
    case RODIMUS_OK: return "ok";
    case RODIMUS_ERR_NULL: return "required pointer is NULL";
    case RODIMUS_ERR_SHAPE: return "invalid shape";
    case RODIMUS_ERR_DTYPE: return "unknown dtype, ingate or struct_size";
    case RODIMUS_ERR_ALIGN: return "pointer not sufficiently aligned";
    case RODIMUS_ERR_SEQLENS: return "invalid cu_seqlens";
    case RODIMUS_ERR_WORKSPACE: return "workspace missing or too small";
    case RODIMUS_ERR_UNSUPPORTED: return "unsupported request";
    case RODIMUS_ERR_CUDA: return "CUDA call failed";
    case RODIMUS_ERR_TIMEOUT: return "bounded device wait ran out";
    default: return "unknown status";
  }
}

int rodimus_version(void) { return 105; }

}  // extern "C"
