// Host-side glue of the C ABI: argument checks, error strings, tensor-map encoding, workspace sizing.
#include <mutex>

#include "common.cuh"

size_t rs_attn_workspace_bytes(const rs_problem* p, int max_kv);
size_t rs_probe_workspace_bytes(const rs_problem* p);
size_t rs_indices_workspace_bytes(const rs_problem* p, const rs_candidate* lib, int n_cand);

extern "C" const char* rs_error_string(int code) {
  switch (code) {
    case RS_OK: return "ok";
    case RS_ERR_INVALID_ARG: return "invalid argument";
    case RS_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (d must be 128; n_keys and segment bounds multiples of 64)";
    case RS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small (see rs_workspace_bytes)";
    case RS_ERR_CUDA: return "CUDA runtime or driver error";
    case RS_ERR_UNSUPPORTED_DEVICE: return "device is not sm_100";
    case RS_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case RS_ERR_NOALLOC_TOO_LARGE:
      return "problem exceeds the built-in scratch of the no-allocation entry point (heads x 128-row tiles > 16384)";
    default: return "unknown error";
  }
}

extern "C" int rs_version(void) { return 100; }

int rs_check_problem(const rs_problem* p) {
  if (p == nullptr || p->seg_bounds == nullptr) return RS_ERR_INVALID_ARG;
  if (p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->n_q_heads % p->n_kv_heads != 0) return RS_ERR_INVALID_ARG;
  if (p->head_dim != RS_HEAD_DIM) return RS_ERR_UNSUPPORTED_SHAPE;
  if (p->n_keys <= 0 || p->n_keys % RS_BLOCK != 0 || p->n_keys > RS_MAX_KEYS) return RS_ERR_UNSUPPORTED_SHAPE;
  if (p->n_segments <= 0 || p->n_segments > RS_MAX_SEGMENTS) return RS_ERR_UNSUPPORTED_SHAPE;
  if (p->seg_bounds[0] != 0 || p->seg_bounds[p->n_segments] != p->n_keys) return RS_ERR_INVALID_ARG;
  for (int s = 0; s < p->n_segments; ++s) {
    const int a = p->seg_bounds[s], b = p->seg_bounds[s + 1];
    if (b <= a) return RS_ERR_INVALID_ARG;
    if (b % RS_BLOCK != 0) return RS_ERR_UNSUPPORTED_SHAPE;
  }
  if ((long long)p->n_q_heads * p->n_keys >= (1ll << 31)) return RS_ERR_UNSUPPORTED_SHAPE;
  return RS_OK;
}

int rs_check_device() {
  static int cached[64];
  static bool init = false;
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!init) { for (int i = 0; i < 64; ++i) cached[i] = 1; init = true; }
  if (dev < 0 || dev >= 64) return RS_ERR_UNSUPPORTED_DEVICE;
  if (cached[dev] == 1) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return RS_ERR_CUDA;
    cached[dev] = (major == 10) ? RS_OK : RS_ERR_UNSUPPORTED_DEVICE;
  }
  return cached[dev];
}

namespace {
struct SideStream {
  std::mutex mu;
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, mid = nullptr;
};
SideStream g_side[64];
thread_local int t_side_dev = -1;   // device whose side stream this thread holds between fork and join
}  // namespace

int rs_side_fork(cudaStream_t main, cudaStream_t* side) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RS_ERR_CUDA;
  if (dev < 0 || dev >= 64) return RS_ERR_UNSUPPORTED_DEVICE;
  SideStream& S = g_side[dev];
  S.mu.lock();
  if (S.stream == nullptr) {
    if (cudaStreamCreateWithFlags(&S.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&S.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&S.join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&S.mid, cudaEventDisableTiming) != cudaSuccess) {
      S.stream = nullptr;
      S.mu.unlock();
      return RS_ERR_CUDA;
    }
  }
  if (cudaEventRecord(S.fork, main) != cudaSuccess || cudaStreamWaitEvent(S.stream, S.fork, 0) != cudaSuccess) {
    S.mu.unlock();
    return RS_ERR_CUDA;
  }
  t_side_dev = dev;
  *side = S.stream;
  return RS_OK;
}

int rs_side_sync_here(cudaStream_t main) {
  if (t_side_dev < 0) return RS_ERR_INVALID_ARG;
  SideStream& S = g_side[t_side_dev];
  return cudaEventRecord(S.mid, S.stream) == cudaSuccess && cudaStreamWaitEvent(main, S.mid, 0) == cudaSuccess ? RS_OK
                                                                                                               : RS_ERR_CUDA;
}

int rs_side_join(cudaStream_t main) {
  if (t_side_dev < 0) return RS_ERR_INVALID_ARG;
  SideStream& S = g_side[t_side_dev];
  t_side_dev = -1;
  const bool ok = cudaEventRecord(S.join, S.stream) == cudaSuccess && cudaStreamWaitEvent(main, S.join, 0) == cudaSuccess;
  S.mu.unlock();
  return ok ? RS_OK : RS_ERR_CUDA;
}

typedef CUresult (*encode_fn_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static encode_fn_t get_encode() {
  static encode_fn_t fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_fn_t>(ptr);
  });
  return fn;
}

static int make_tmap_2d(CUtensorMap* out, CUtensorMapDataType dt, size_t esize, const void* base, uint64_t rows,
                        uint64_t cols, uint32_t box_rows, uint32_t box_cols) {
  encode_fn_t enc = get_encode();
  if (enc == nullptr) return RS_ERR_CUDA;
  if (((uintptr_t)base & 15) != 0) return RS_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * esize};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? RS_OK : RS_ERR_CUDA;
}

int rs_make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols) {
  return make_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, rows, cols, box_rows, box_cols);
}
int rs_make_tmap_f32_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                        uint32_t box_cols) {
  return make_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, rows, cols, box_rows, box_cols);
}

extern "C" int rs_workspace_bytes(const rs_problem* p, const rs_candidate* lib, int n_cand, size_t* bytes) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (bytes == nullptr || n_cand < 0 || n_cand > RS_MAX_CANDIDATES || (n_cand > 0 && lib == nullptr))
    return RS_ERR_INVALID_ARG;
  int max_kv = 0;
  for (int c = 0; c < n_cand; ++c)
    if (lib[c].pattern == RS_VERTICAL_SLASH && lib[c].b0 > max_kv) max_kv = lib[c].b0;
  if (max_kv > p->n_keys) max_kv = p->n_keys;
  size_t need = rs_attn_workspace_bytes(p, max_kv);
  size_t b = rs_probe_workspace_bytes(p);
  if (b > need) need = b;
  b = rs_indices_workspace_bytes(p, lib, n_cand);
  if (b > need) need = b;
  *bytes = rs_align_up(need, 256);
  return RS_OK;
}

// ------------------------------------------------------------------------------------------ self test of the bounded wait
namespace {
__global__ void rs_selftest_wait_kernel(int32_t* status, unsigned int limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  __syncthreads();
  // nothing ever arrives on this barrier: the wait has to give up by itself and the kernel has to end normally
  if (threadIdx.x == 0 && !mbar_wait(smem_u32(&bar), 0, &abort_flag, limit)) rs_report(status, RS_ERR_TIMEOUT, 99);
}
}  // namespace

extern "C" int rs_selftest_wait_timeout(int32_t* status, unsigned int poll_limit, void* stream) {
  if (status == nullptr || poll_limit == 0 || poll_limit > (1u << 20)) return RS_ERR_INVALID_ARG;
  rs_selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(status, poll_limit);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------ query mixture of Eq. 3 (host)
extern "C" int rs_mixture_rows(int q0, int q1, int r_recent, int r_uniform, int r_boundary, int32_t* rows) {
  if (rows == nullptr || q0 < 0 || q1 <= q0 || r_recent < 0 || r_uniform < 0 || r_boundary < 0) return RS_ERR_INVALID_ARG;
  const long long span = (long long)(q1 - q0) - r_recent - r_boundary;
  if (span < r_uniform) return RS_ERR_UNSUPPORTED_SHAPE;       // the three groups would overlap
  int at = 0;
  for (int k = 0; k < r_recent; ++k) rows[at++] = q1 - r_recent + k;
  for (int k = 0; k < r_uniform; ++k) rows[at++] = q0 + r_boundary + (int)(((2ll * k + 1) * span) / (2ll * r_uniform));
  for (int k = 0; k < r_boundary; ++k) rows[at++] = q0 + k;
  return RS_OK;
}

extern "C" int rs_mixture_runs(int q0, int q1, int32_t* run_starts) {
  if (run_starts == nullptr || q0 < 0 || q1 - q0 < RS_PROBE_ROWS || (q1 - q0) % 16 != 0) return RS_ERR_INVALID_ARG;
  const int units = (q1 - q0) / 16;
  run_starts[0] = q0;
  run_starts[1] = q0 + 16 * (units / 3);
  run_starts[2] = q0 + 16 * ((2 * units) / 3);
  run_starts[3] = q1 - 16;
  return RS_OK;
}
