// C-ABI entry points (see include/smartmem.h).
#include <atomic>
#include <mutex>
#include <set>
#include <utility>
#include <vector>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "plan.hpp"
#include "ptx.cuh"

#define EXPORT extern "C" __attribute__((visibility("default")))

namespace smartmem {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches += n; }

static std::mutex g_prof_mu;
static bool g_prof_on = false;
static std::vector<cudaEvent_t> g_prof_ev;
static std::vector<const char*> g_prof_names;
void profile_tick(const char* name, cudaStream_t st) {
  if (!g_prof_on) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  cudaEvent_t e;
  if (cudaEventCreate(&e) != cudaSuccess) return;
  cudaEventRecord(e, st);
  g_prof_ev.push_back(e);
  g_prof_names.push_back(name);
}

// Status block of the device: word 0 the status, words 2-3 the limit (ns) of every bounded device-side wait.
__device__ __align__(16) int g_status_word[4];

// Both caches below are per device: the address of a __device__ symbol and a kernel's attributes belong to the
// context of the device that was current when they were looked up or set.
static constexpr int kMaxDevices = 64;
static std::mutex g_dev_mu;
static int* g_status_ptr[kMaxDevices] = {nullptr};

int* device_status_ptr() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lk(g_dev_mu);
  if (!g_status_ptr[dev]) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_status_word) != cudaSuccess || !q) return nullptr;
    const unsigned long long limit = smartmem::ptx::kWaitLimitNs;
    if (cudaMemset(q, 0, 4 * sizeof(int)) != cudaSuccess) return nullptr;
    if (cudaMemcpy((int*)q + 2, &limit, sizeof(limit), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    g_status_ptr[dev] = (int*)q;
  }
  return g_status_ptr[dev];
}

static std::set<std::pair<int, const void*>> g_smem_configured;

int ensure_max_dynamic_smem(const void* kernel, int bytes, int carveout) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return SMARTMEM_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_dev_mu);
  const auto key = std::make_pair(dev, kernel);
  if (g_smem_configured.count(key)) return SMARTMEM_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return SMARTMEM_ERR_CUDA;
  if (carveout >= 0) cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, carveout);
  g_smem_configured.insert(key);
  return SMARTMEM_OK;
}

}  // namespace smartmem

using namespace smartmem;

EXPORT int smartmem_profile_begin(void) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  for (cudaEvent_t e : g_prof_ev) cudaEventDestroy(e);
  g_prof_ev.clear();
  g_prof_names.clear();
  g_prof_on = true;
  return SMARTMEM_OK;
}

EXPORT int smartmem_profile_end(void* cuda_stream, float* kernel_ms, char* kernel_names, int32_t names_stride,
                                int32_t max_kernels, int32_t* n_kernels) {
  if (!kernel_ms || !kernel_names || !n_kernels || max_kernels < 1 || names_stride < 8) return SMARTMEM_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  profile_tick("end", st);
  std::lock_guard<std::mutex> lk(g_prof_mu);
  g_prof_on = false;
  int rs = cudaStreamSynchronize(st) == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
  int n = 0;
  for (size_t i = 0; i + 1 < g_prof_ev.size() && n < max_kernels; ++i, ++n) {
    float ms = 0.f;
    if (rs == SMARTMEM_OK) cudaEventElapsedTime(&ms, g_prof_ev[i], g_prof_ev[i + 1]);
    kernel_ms[n] = ms;
    const char* nm = g_prof_names[i];
    int k = 0;
    while (nm[k] && k < names_stride - 1) { kernel_names[n * names_stride + k] = nm[k]; ++k; }
    kernel_names[n * names_stride + k] = 0;
  }
  for (cudaEvent_t e : g_prof_ev) cudaEventDestroy(e);
  g_prof_ev.clear();
  g_prof_names.clear();
  *n_kernels = n;
  return rs;
}

EXPORT int64_t smartmem_launch_count(void) { return g_launches.load(); }

EXPORT int smartmem_last_device_status(void* cuda_stream, int32_t* status) {
  if (!status) return SMARTMEM_ERR_INVALID_ARG;
  int* p = device_status_ptr();
  if (!p) return SMARTMEM_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int v = 0;
  if (cudaMemcpyAsync(&v, p, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SMARTMEM_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SMARTMEM_ERR_CUDA;
  if (v != 0) cudaMemsetAsync(p, 0, sizeof(int), st);
  *status = v;
  return SMARTMEM_OK;
}

namespace {
// A wait that nothing will ever satisfy, through the same bounded wait the kernels use: one warp waits on
// a barrier that expects an arrival which never comes.  The wait gives up after the device's wait limit,
// raises SMARTMEM_ERR_TIMEOUT in the status word and the kernel returns normally.
__global__ void selftest_wait_kernel(int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  ptx::mbar_wait(&bar, 0, &abort_flag, status);
}
}  // namespace

extern "C" int smartmem_set_wait_limit_ns(uint64_t limit_ns) {
  int* p = device_status_ptr();
  if (!p) return SMARTMEM_ERR_CUDA;
  if (limit_ns == 0 || limit_ns > 60000000000ull) return SMARTMEM_ERR_INVALID_ARG;
  const unsigned long long v = limit_ns;
  if (cudaDeviceSynchronize() != cudaSuccess) return SMARTMEM_ERR_CUDA;       // no kernel reads the limit while it changes
  return cudaMemcpy(p + 2, &v, sizeof(v), cudaMemcpyHostToDevice) == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

extern "C" int smartmem_selftest_bounded_wait(void* cuda_stream) {
  int* p = device_status_ptr();
  if (!p) return SMARTMEM_ERR_CUDA;
  selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(p);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

namespace {

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

bool make_devseq(const SeqProgram& sp, DevSeq* out) {
  if (sp.stages.size() > (size_t)kSeqMaxStages || sp.src_shape.size() > (size_t)kSeqMaxDims) return false;
  memset(out, 0, sizeof(*out));
  out->n_stages = (int)sp.stages.size();
  out->n_src = (int)sp.src_shape.size();
  for (int k = 0; k < out->n_src; ++k) {
    out->src_shape[k] = sp.src_shape[k];
    out->src_stride[k] = sp.src_stride[k];
  }
  for (int i = 0; i < out->n_stages; ++i) {
    const SeqStage& a = sp.stages[i];
    DevSeqStage& d = out->st[i];
    if (a.in_shape.size() > (size_t)kSeqMaxDims || a.out_shape.size() > (size_t)kSeqMaxDims) return false;
    d.kind = a.kind; d.n_in = (int)a.in_shape.size(); d.n_out = (int)a.out_shape.size();
    d.axis = a.axis;
    if (a.shift > (1ll << 30) || a.shift < -(1ll << 30)) return false;
    d.shift = (int)a.shift;
    for (int k = 0; k < d.n_in; ++k) { if (a.in_shape[k] >= (1ll << 31)) return false; d.in_shape[k] = (int)a.in_shape[k]; }
    for (int k = 0; k < d.n_out; ++k) { if (a.out_shape[k] >= (1ll << 31)) return false; d.out_shape[k] = (int)a.out_shape[k]; }
    for (size_t k = 0; k < a.perm.size(); ++k) d.aux[k] = a.perm[k];
    for (size_t k = 0; k < a.start.size(); ++k) d.aux[k] = (int)a.start[k];
  }
  return true;
}

}  // namespace

EXPORT int smartmem_run_chain(const smartmem_plan_t* plan, const void* const* inputs, void* const* outputs,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!plan || !inputs || !outputs || !outputs[0]) return SMARTMEM_ERR_INVALID_ARG;
  for (int i = 0; i < plan->n_inputs; ++i) {
    if (!inputs[i]) return SMARTMEM_ERR_INVALID_ARG;
    if (!aligned16(inputs[i])) return SMARTMEM_ERR_ALIGNMENT;
  }
  if (!aligned16(outputs[0]) || !aligned16(workspace)) return SMARTMEM_ERR_ALIGNMENT;
  if (plan->workspace_bytes > workspace_bytes || (plan->workspace_bytes && !workspace)) return SMARTMEM_ERR_WORKSPACE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return SMARTMEM_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  auto buf = [&](int ref) -> void* {
    if (ref >= 0) return const_cast<void*>(inputs[ref]);
    if (ref == -1) return outputs[0];
    return (char*)workspace + plan->slot_offset[-2 - ref];
  };
  for (const Step& s : plan->steps) {
    const int esz = s.dtype == SMARTMEM_F32 ? 4 : 2;
    int rc = SMARTMEM_OK;
    if (s.kind == STEP_COPY) {
      if (s.map[0].klass == 3 || (plan->mode == SMARTMEM_ELIMINATE_NAIVE && !s.is_layout_copy)) {
        DevSeq q;
        if (!make_devseq(s.seq[0], &q)) return SMARTMEM_ERR_UNSUPPORTED;
        rc = launch_copy_seq(q, s.map[0].n_elements, esz, buf(s.src[0]), buf(s.dst), st);
      } else {
        rc = launch_copy_map(s.map[0], esz, buf(s.src[0]), buf(s.dst), st, s.placement);
      }
    } else if (s.kind == STEP_LINEAR || s.kind == STEP_BMM_NT) {
      if (s.dtype != SMARTMEM_BF16) return SMARTMEM_ERR_UNSUPPORTED;
      TcOperand A, B;
      rc = tc_operand_from_map(s.map[0], s.n_batch_atoms[0], s.n_row_atoms[0], buf(s.src[0]), &A);
      if (rc != SMARTMEM_OK) return rc;
      if (s.kind == STEP_LINEAR) {
        B = tc_operand_plain(inputs[s.weight], s.N, s.K, s.K);
      } else {
        rc = tc_operand_from_map(s.map[1], s.n_batch_atoms[1], s.n_row_atoms[1], buf(s.src[1]), &B);
        if (rc != SMARTMEM_OK) return rc;
      }
      TcEpilogue ep;
      memset(&ep, 0, sizeof(ep));
      ep.out = buf(s.dst);
      ep.ldc = s.N;
      ep.out_batch_stride = s.M * s.N;
      rc = launch_gemm_tc(A, B, ep, s.batch, s.M, s.N, s.K, st);
    } else if (s.kind == STEP_NORM) {
      rc = launch_layernorm_map(s.dtype, buf(s.src[0]), buf(s.dst), inputs[s.weight], inputs[s.weight2], s.eps, s.map[0],
                                (int)s.K, st);
    } else {
      rc = SMARTMEM_ERR_UNSUPPORTED;
    }
    if (rc != SMARTMEM_OK) return rc;
  }
  return SMARTMEM_OK;
}

