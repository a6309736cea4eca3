// Attention-output error certificate, Eq. 5: ||aV - a~V||_2 <= 2 (1 - m) V_max with the retained mass
// m = exp(lse_sel - lse_full) taken from the two log-sum-exps of a row.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(256)
rs_certificate_kernel(int n_keys, int group, const float* lse_sel, const float* lse_full, const int32_t* rows, int n_rows,
                      const float* vmax_head, const float* onorm, float delta_q, float* m_row, float* cert_row,
                      float* cert_tight, float* m_head, float* cert_head, int32_t* status) {
  __shared__ double s_sum[8];
  __shared__ float s_max[8];
  __shared__ int s_ok;
  if (threadIdx.x == 0) s_ok = 0;
  __syncthreads();
  const int h = blockIdx.x;
  const float vmax = vmax_head[h / group];
  double sum = 0.0;
  float cmax = 0.f;
  int n_ok = 0;
  for (int r = threadIdx.x; r < n_rows; r += blockDim.x) {
    const int row = rows[r];
    const size_t dst = (size_t)h * n_rows + r;
    if (row < 0 || row >= n_keys) {          // a bad row id is reported, never dereferenced
      rs_report(status, RS_ERR_INVALID_ARG, 60);
      const float nan = __int_as_float(0x7fc00000);
      if (m_row) m_row[dst] = nan;
      if (cert_row) cert_row[dst] = nan;
      if (cert_tight && onorm) cert_tight[dst] = nan;
      continue;
    }
    ++n_ok;
    const size_t src = (size_t)h * n_keys + row;
    const float m = fminf(1.0f, expf(lse_sel[src] - lse_full[dst]));
    const float cert = 2.0f * (1.0f - m) * vmax;
    if (m_row) m_row[dst] = m;
    if (cert_row) cert_row[dst] = cert;
    if (cert_tight && onorm) cert_tight[dst] = (1.0f - m) * (vmax + onorm[src]);
    sum += (double)m;
    cmax = fmaxf(cmax, cert);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, off);
    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, off));
  }
  if ((threadIdx.x & 31) == 0) { s_sum[threadIdx.x >> 5] = sum; s_max[threadIdx.x >> 5] = cmax; }
  if (n_ok > 0) atomicAdd(&s_ok, n_ok);
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    float mx = 0.f;
    for (int w = 0; w < 8; ++w) { t += s_sum[w]; mx = fmaxf(mx, s_max[w]); }
    const double mh = t / (double)max(1, s_ok);
    const double m_low = fmax(0.0, mh - (double)delta_q);
    if (m_head) m_head[h] = (float)mh;
    if (cert_head) { cert_head[2 * h] = (float)(2.0 * (1.0 - m_low) * (double)vmax); cert_head[2 * h + 1] = mx; }
  }
}

}  // namespace

extern "C" int rs_certificate(int n_q_heads, int n_kv_heads, int n_keys, const float* lse_sel, const float* lse_full,
                              const int32_t* rows, int n_rows, const float* vmax_head, const float* onorm,
                              float delta_q, float* m_row, float* cert_row, float* cert_tight, float* m_head,
                              float* cert_head, int32_t* status, void* stream_) {
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0 || n_keys <= 0 || n_rows <= 0 || !lse_sel || !lse_full || !rows || !vmax_head)
    return RS_ERR_INVALID_ARG;
  rs_certificate_kernel<<<n_q_heads, 256, 0, (cudaStream_t)stream_>>>(n_keys, n_q_heads / n_kv_heads, lse_sel, lse_full, rows, n_rows, vmax_head,
                                                                     onorm, delta_q, m_row, cert_row, cert_tight, m_head,
                                                                     cert_head, status);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------------------------
// Offline calibration helpers (Section 3.5): row-wise output error of a dense audit, and the monotone predictor e of
// Eq. 4 evaluated for every (item, candidate) from the probe descriptors and the candidate statistics.
namespace {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// one warp per row: lane l handles dimensions l, l + 32, l + 64, l + 96; fixed-order butterfly
template <typename T>
__global__ void __launch_bounds__(256)
rs_output_error_kernel(long long n_rows, const T* __restrict__ a, const T* __restrict__ b, float* err, float* norm_a) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int lane = threadIdx.x & 31;
  float d2 = 0.f, a2 = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float x = to_f32(a[row * RS_HEAD_DIM + lane + 32 * k]), y = to_f32(b[row * RS_HEAD_DIM + lane + 32 * k]);
    d2 = fmaf(x - y, x - y, d2);
    a2 = fmaf(x, x, a2);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    d2 += __shfl_xor_sync(0xffffffffu, d2, off);
    a2 += __shfl_xor_sync(0xffffffffu, a2, off);
  }
  if (lane == 0) {
    if (err) err[row] = sqrtf(d2);
    if (norm_a) norm_a[row] = sqrtf(a2);
  }
}

struct RegArgs {
  int n_items, n_cand, Hq, n_bp;
  int seg_bounds[RS_MAX_SEGMENTS + 1];
  rs_candidate lib[RS_MAX_CANDIDATES];
  double w[6];
  double bp_z[64], bp_e[64];
};

__global__ void rs_regressor_kernel(const __grid_constant__ RegArgs A, const rs_cand_stats* stats, const float* descr,
                                    double* e_out) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= A.n_items * A.n_cand) return;
  const int item = idx / A.n_cand, c = idx - item * A.n_cand;
  if (A.lib[c].pattern == RS_DENSE) { e_out[idx] = 0.0; return; }
  const rs_cand_stats& st = stats[idx];
  const int s = item / A.Hq;
  const long long q0 = A.seg_bounds[s], q1 = A.seg_bounds[s + 1];
  const double dense_pairs = (double)((q1 * (q1 + 1) - q0 * (q0 + 1)) / 2);
  unsigned long long tot = 0;
  double mx = 0.0, mn = 2.0;
  for (int g = 0; g < RS_PROBE_GROUPS; ++g) {
    tot += st.cov_fx[g];
    const double mg = (double)st.cov_fx[g] / 68719476736.0;     // 16 rows * 2^32
    mx = fmax(mx, mg);
    mn = fmin(mn, mg);
  }
  const double m_hat = (double)tot / 274877906944.0;             // 64 rows * 2^32
  const double f[6] = {__dsub_rn(1.0, m_hat), __dsub_rn(mx, mn), (double)descr[item * 4 + 0],
                       __dsub_rn(1.0, (double)descr[item * 4 + 1]), __dsub_rn(1.0, (double)descr[item * 4 + 2]),
                       __dsub_rn(1.0, __ddiv_rn((double)st.pairs, dense_pairs))};
  double z = 0.0;
  for (int k = 0; k < 6; ++k) z = __dadd_rn(z, __dmul_rn(A.w[k], f[k]));
  double e = 0.0;
  for (int k = 0; k < A.n_bp; ++k) if (A.bp_z[k] <= z) e = A.bp_e[k];
  e_out[idx] = e;
}

}  // namespace

extern "C" int rs_output_error(long long n_rows, const void* Oa, const void* Ob, int o_dtype, float* err, float* norm_a,
                               int32_t* status, void* stream_) {
  (void)status;
  if (n_rows <= 0 || !Oa || !Ob || (!err && !norm_a) || (o_dtype != 0 && o_dtype != 1)) return RS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const unsigned grid = (unsigned)((n_rows + 7) / 8);
  if (o_dtype == 1)
    rs_output_error_kernel<float><<<grid, 256, 0, stream>>>(n_rows, (const float*)Oa, (const float*)Ob, err, norm_a);
  else
    rs_output_error_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(n_rows, (const __nv_bfloat16*)Oa, (const __nv_bfloat16*)Ob, err, norm_a);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

extern "C" int rs_regressor_eval(const rs_problem* p, const rs_candidate* lib, int n_cand, const rs_cand_stats* stats,
                                 const float* descr, const double* w, const double* bp_z, const double* bp_e, int n_bp,
                                 double* e_out, int32_t* status, void* stream_) {
  (void)status;
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!lib || n_cand <= 0 || n_cand > RS_MAX_CANDIDATES || !stats || !descr || !w || !e_out) return RS_ERR_INVALID_ARG;
  if (n_bp < 0 || n_bp > 64 || (n_bp > 0 && (!bp_z || !bp_e))) return RS_ERR_INVALID_ARG;
  for (int k = 0; k < 6; ++k) if (!(w[k] >= 0.0)) return RS_ERR_INVALID_ARG;
  for (int k = 1; k < n_bp; ++k) if (!(bp_z[k] > bp_z[k - 1]) || !(bp_e[k] >= bp_e[k - 1])) return RS_ERR_INVALID_ARG;
  RegArgs A{};
  A.n_items = p->n_segments * p->n_q_heads; A.n_cand = n_cand; A.Hq = p->n_q_heads; A.n_bp = n_bp;
  for (int s = 0; s <= p->n_segments; ++s) A.seg_bounds[s] = p->seg_bounds[s];
  for (int c = 0; c < n_cand; ++c) A.lib[c] = lib[c];
  for (int k = 0; k < 6; ++k) A.w[k] = w[k];
  for (int k = 0; k < n_bp; ++k) { A.bp_z[k] = bp_z[k]; A.bp_e[k] = bp_e[k]; }
  const int n = A.n_items * n_cand;
  rs_regressor_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream_>>>(A, stats, descr, e_out);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
