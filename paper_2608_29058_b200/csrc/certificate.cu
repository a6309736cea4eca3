// Attention-output error certificate, Eq. 5: ||aV - a~V||_2 <= 2 (1 - m) V_max with the retained mass
// m = exp(lse_sel - lse_full) taken from the two log-sum-exps of a row.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(256)
rs_certificate_kernel(int n_keys, int group, const float* lse_sel, const float* lse_full, const int32_t* rows, int n_rows,
                      const float* vmax_head, const float* onorm, float delta_q, float* m_row, float* cert_row,
                      float* cert_tight, float* m_head, float* cert_head) {
  __shared__ double s_sum[8];
  __shared__ float s_max[8];
  const int h = blockIdx.x;
  const float vmax = vmax_head[h / group];
  double sum = 0.0;
  float cmax = 0.f;
  for (int r = threadIdx.x; r < n_rows; r += blockDim.x) {
    const size_t src = (size_t)h * n_keys + rows[r];
    const size_t dst = (size_t)h * n_rows + r;
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
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    float mx = 0.f;
    for (int w = 0; w < 8; ++w) { t += s_sum[w]; mx = fmaxf(mx, s_max[w]); }
    const double mh = t / (double)n_rows;
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
  (void)status;
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0 || n_keys <= 0 || n_rows <= 0 || !lse_sel || !lse_full || !rows || !vmax_head)
    return RS_ERR_INVALID_ARG;
  rs_certificate_kernel<<<n_q_heads, 256, 0, (cudaStream_t)stream_>>>(n_keys, n_q_heads / n_kv_heads, lse_sel, lse_full, rows, n_rows, vmax_head,
                                                                     onorm, delta_q, m_row, cert_row, cert_tight, m_head,
                                                                     cert_head);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
