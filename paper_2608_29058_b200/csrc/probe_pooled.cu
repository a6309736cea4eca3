// Eq. 3 in its general form (Section 3.2): r sampled query rows of every head against keys pooled over blocks of
// width g, soft-maxed over the visible blocks, reduced to column / diagonal block mass per row subset and to the
// three descriptors (entropy, local-band concentration, agreement between the first two subsets).
//
// A key block is visible to row i when its first key is <= i and is pooled (arithmetic mean, fp32) over its visible
// keys only.  With r <= 64 rows and g >= 8 the products are small (about 1 GFLOP per layer at g = 64, n = 128K), so
// they run on the FMA pipes: three streaming kernels, no tensor cores.
#include "common.cuh"

namespace {

constexpr int kMaxRows = 64;       // probe rows per (segment, head)
constexpr int kSig = 18;           // signature bins: [key block 0] + [relative block offsets 0..15] + [rest]
constexpr int kLocalBand = 1024;
constexpr int kKB = 8;             // pooled key blocks per inner iteration of the logits kernel
constexpr int kMaxSub = 4;

struct PoolParams {
  int n, Hq, Hkv, group, n_seg, r, g, n_sub;
  int seg_bounds[RS_MAX_SEGMENTS + 1];
  int sub_bounds[kMaxSub + 1];
  const __nv_bfloat16* Q;
  const __nv_bfloat16* K;
  const int32_t* rows;   // [n_seg][r]
  float* A;              // [n_seg][Hq][r][n / g]: logits, then probabilities
  float* lse;            // [n_seg][Hq][r]
  float* colmass;        // [n_seg][Hq][n_sub][n / g]
  float* diagmass;       // [n_seg][Hq][n_sub][n / g]
  float* descr;          // [n_seg][Hq][4]: entropy, local-band mass, agreement, mean number of visible blocks
  float* rowstat;        // [n_seg][Hq][r][2 + kSig] scratch: entropy, local mass, signature of each row
  float scale;
};

// Logits of every probe row of the (up to four) query heads of one KV head against the fully visible key blocks.
// Block = 256 threads = 4 head slots x 64 row slots; Q^T sits in shared memory as [dim][row] so that a warp reads
// consecutive rows; each iteration pools kKB key blocks and every thread accumulates kKB dot products.
__global__ void __launch_bounds__(256)
rs_pp_logits_kernel(PoolParams P, int blocks_per_cta) {
  extern __shared__ uint8_t smem_raw[];
  __nv_bfloat16* qT = reinterpret_cast<__nv_bfloat16*>(smem_raw);                   // [128][256]
  float* pooled = reinterpret_cast<float*>(smem_raw + 128 * 256 * 2);              // [kKB][128]
  const int s = blockIdx.y / P.Hkv, gk = blockIdx.y % P.Hkv;
  const int q1 = P.seg_bounds[s + 1];
  const int nbg = P.n / P.g, nbg_seg = q1 / P.g;
  const int tid = threadIdx.x;
  const int hh = tid >> 6, t = tid & 63;
  const bool live = hh < P.group && t < P.r;
  const int h = gk * P.group + hh;
  const int i = live ? P.rows[s * P.r + t] : -1;
  const int kb_d = live ? i / P.g : -1;            // the diagonal block: pooled over a prefix, done by the softmax kernel
  for (int e = tid; e < 128 * 256; e += 256) {
    const int row = e >> 7, dim = e & 127;         // consecutive threads read consecutive dims of one row
    const int rh = row >> 6, rt = row & 63;
    __nv_bfloat16 v = __float2bfloat16(0.f);
    if (rh < P.group && rt < P.r) {
      const int ri = P.rows[s * P.r + rt];
      v = P.Q[((size_t)(gk * P.group + rh) * P.n + ri) * RS_HEAD_DIM + dim];
    }
    qT[dim * 256 + row] = v;
  }
  __syncthreads();
  const int kb_begin = blockIdx.x * blocks_per_cta;
  const int kb_end = min(nbg_seg, kb_begin + blocks_per_cta);
  float* out = live ? P.A + (((size_t)s * P.Hq + h) * P.r + t) * (size_t)nbg : nullptr;
  const float inv_g = 1.0f / (float)P.g;
  for (int kb0 = kb_begin; kb0 < kb_end; kb0 += kKB) {
    // pooled[b][dim] = mean of the g keys of block kb0 + b (threads: dim = tid & 127, blocks b = tid >> 7, +2, ..)
    for (int b = tid >> 7; b < kKB; b += 2) {
      const int kb = kb0 + b;
      float acc = 0.f;
      if (kb < kb_end) {
        const __nv_bfloat16* src = P.K + ((size_t)gk * P.n + (size_t)kb * P.g) * RS_HEAD_DIM + (tid & 127);
        for (int j = 0; j < P.g; ++j) acc += __bfloat162float(src[(size_t)j * RS_HEAD_DIM]);
      }
      pooled[b * 128 + (tid & 127)] = acc * inv_g;
    }
    __syncthreads();
    float acc[kKB];
#pragma unroll
    for (int b = 0; b < kKB; ++b) acc[b] = 0.f;
#pragma unroll 4
    for (int dim = 0; dim < 128; ++dim) {
      const float qv = __bfloat162float(qT[dim * 256 + tid]);
#pragma unroll
      for (int b = 0; b < kKB; ++b) acc[b] = fmaf(qv, pooled[b * 128 + dim], acc[b]);
    }
    if (live) {
#pragma unroll
      for (int b = 0; b < kKB; ++b) {
        const int kb = kb0 + b;
        if (kb < kb_end && kb < kb_d) out[kb] = acc[b] * P.scale;
      }
    }
    __syncthreads();
  }
}

__device__ __forceinline__ float block_reduce_sum(float v, float* red) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
  return t;
}
__device__ __forceinline__ float block_reduce_max(float v, float* red) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = -INFINITY;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t = fmaxf(t, red[w]);
  return t;
}

// One block per probe row: the diagonal block's logit (prefix pooling), soft-max over the visible blocks in place,
// the row's entropy, local-band mass and signature.
__global__ void __launch_bounds__(256)
rs_pp_softmax_kernel(PoolParams P) {
  __shared__ float red[8];
  __shared__ float sig[kSig];
  __shared__ float kpre[128];
  const int t = blockIdx.x;
  const int s = blockIdx.y / P.Hq, h = blockIdx.y % P.Hq;
  const int gk = h / P.group;
  const int nbg = P.n / P.g;
  const int tid = threadIdx.x;
  const int i = P.rows[s * P.r + t];
  const int kb_d = i / P.g;
  float* a = P.A + (((size_t)s * P.Hq + h) * P.r + t) * (size_t)nbg;
  // diagonal block: mean of keys kb_d * g .. i, then the dot product with the row
  if (tid < 128) {
    const __nv_bfloat16* src = P.K + ((size_t)gk * P.n + (size_t)kb_d * P.g) * RS_HEAD_DIM + tid;
    const int cnt = i - kb_d * P.g + 1;
    float acc = 0.f;
    for (int j = 0; j < cnt; ++j) acc += __bfloat162float(src[(size_t)j * RS_HEAD_DIM]);
    kpre[tid] = acc / (float)cnt;
  }
  if (tid < kSig) sig[tid] = 0.f;
  __syncthreads();
  float part = 0.f;
  if (tid < 128) part = kpre[tid] * __bfloat162float(P.Q[((size_t)h * P.n + i) * RS_HEAD_DIM + tid]);
  const float ld = block_reduce_sum(part, red) * P.scale;
  if (tid == 0) a[kb_d] = ld;
  __syncthreads();
  const int vis = kb_d + 1;
  float mx = -INFINITY;
  for (int kb = tid; kb < vis; kb += 256) mx = fmaxf(mx, a[kb]);
  mx = block_reduce_max(mx, red);
  float sum = 0.f;
  for (int kb = tid; kb < vis; kb += 256) sum += __expf(a[kb] - mx);
  sum = block_reduce_sum(sum, red);
  const float lse = mx + __logf(sum);
  float es = 0.f, loc = 0.f;
  float sg_local = 0.f, sg_zero = 0.f, sg_rest = 0.f;
  for (int kb = tid; kb < nbg; kb += 256) {
    float pv = 0.f;
    if (kb < vis) {
      const float sv = a[kb];
      pv = __expf(sv - lse);
      es += pv * sv;
      if (i - kb * P.g < kLocalBand) loc += pv;
      const int delta = kb_d - kb;
      if (delta < kSig - 2) atomicAdd(&sig[1 + delta], pv);
      else if (kb == 0) sg_zero += pv;
      else sg_rest += pv;
    }
    a[kb] = pv;
  }
  (void)sg_local;
  es = block_reduce_sum(es, red);
  loc = block_reduce_sum(loc, red);
  sg_zero = block_reduce_sum(sg_zero, red);
  sg_rest = block_reduce_sum(sg_rest, red);
  __syncthreads();
  float* rs_ = P.rowstat + (((size_t)s * P.Hq + h) * P.r + t) * (2 + kSig);
  if (tid == 0) {
    P.lse[((size_t)s * P.Hq + h) * P.r + t] = lse;
    const float H = lse - es;                                   // -sum a log a = lse - E[s]
    rs_[0] = fmaxf(0.f, H) / __logf((float)max(2, vis));
    rs_[1] = loc;
    rs_[2] = sg_zero;
    rs_[2 + kSig - 1] = sg_rest;
  }
  if (tid >= 1 && tid < kSig - 1) rs_[2 + tid] = sig[tid];
}

// Column / diagonal block mass per subset, and (block 0 of every head) the three descriptors.
__global__ void __launch_bounds__(256)
rs_pp_reduce_kernel(PoolParams P) {
  const int s = blockIdx.y / P.Hq, h = blockIdx.y % P.Hq;
  const int nbg = P.n / P.g;
  const int x = blockIdx.x * 256 + threadIdx.x;
  const size_t head = (size_t)s * P.Hq + h;
  const float* a = P.A + head * P.r * (size_t)nbg;
  if (x < nbg) {
    for (int sb = 0; sb < P.n_sub; ++sb) {
      float col = 0.f, dg = 0.f;
      for (int t = P.sub_bounds[sb]; t < P.sub_bounds[sb + 1]; ++t) {
        col += a[(size_t)t * nbg + x];
        const int kb = P.rows[s * P.r + t] / P.g - x;            // x read as a relative block offset
        if (kb >= 0) dg += a[(size_t)t * nbg + kb];
      }
      P.colmass[(head * P.n_sub + sb) * (size_t)nbg + x] = col;
      P.diagmass[(head * P.n_sub + sb) * (size_t)nbg + x] = dg;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < 32) {
    const int lane = threadIdx.x;
    const float* rs_ = P.rowstat + head * P.r * (2 + kSig);
    float ent = 0.f, loc = 0.f, vis = 0.f;
    for (int t = lane; t < P.r; t += 32) {
      ent += rs_[t * (2 + kSig)];
      loc += rs_[t * (2 + kSig) + 1];
      vis += (float)(P.rows[s * P.r + t] / P.g + 1);
    }
    float tv = 0.f;
    if (P.n_sub >= 2 && lane < kSig) {
      float s0 = 0.f, s1 = 0.f;
      for (int t = P.sub_bounds[0]; t < P.sub_bounds[1]; ++t) s0 += rs_[t * (2 + kSig) + 2 + lane];
      for (int t = P.sub_bounds[1]; t < P.sub_bounds[2]; ++t) s1 += rs_[t * (2 + kSig) + 2 + lane];
      tv = fabsf(s0 / (float)max(1, P.sub_bounds[1] - P.sub_bounds[0]) - s1 / (float)max(1, P.sub_bounds[2] - P.sub_bounds[1]));
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      ent += __shfl_xor_sync(0xffffffffu, ent, off);
      loc += __shfl_xor_sync(0xffffffffu, loc, off);
      vis += __shfl_xor_sync(0xffffffffu, vis, off);
      tv += __shfl_xor_sync(0xffffffffu, tv, off);
    }
    if (lane == 0) {
      float* d = P.descr + head * 4;
      d[0] = ent / (float)P.r;
      d[1] = loc / (float)P.r;
      d[2] = 1.0f - 0.5f * tv;
      d[3] = vis / (float)P.r;
    }
  }
}

}  // namespace

extern "C" int rs_probe_pooled_scratch_floats(const rs_problem* p, int r, size_t* n_floats) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (r < 1 || r > kMaxRows || n_floats == nullptr) return RS_ERR_INVALID_ARG;
  *n_floats = (size_t)p->n_segments * p->n_q_heads * r * (2 + kSig);
  return RS_OK;
}

extern "C" int rs_probe_pooled(const rs_problem* p, const void* Q, const void* K, const int32_t* rows, int r, int g,
                               const int32_t* sub_bounds, int n_sub, float* A, float* lse, float* colmass,
                               float* diagmass, float* descr, float* scratch, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !K || !rows || !sub_bounds || !A || !lse || !colmass || !diagmass || !descr || !scratch) return RS_ERR_INVALID_ARG;
  if (r < 1 || r > kMaxRows || n_sub < 1 || n_sub > kMaxSub) return RS_ERR_INVALID_ARG;
  if (g < 1 || g > RS_BLOCK || RS_BLOCK % g != 0) return RS_ERR_UNSUPPORTED_SHAPE;
  if (p->n_q_heads / p->n_kv_heads > 4) return RS_ERR_UNSUPPORTED_SHAPE;
  if (sub_bounds[0] != 0 || sub_bounds[n_sub] != r) return RS_ERR_INVALID_ARG;
  for (int i = 0; i < n_sub; ++i) if (sub_bounds[i + 1] <= sub_bounds[i]) return RS_ERR_INVALID_ARG;
  rc = rs_check_device();
  if (rc != RS_OK) return rc;
  (void)status;
  cudaStream_t stream = (cudaStream_t)stream_;
  PoolParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = P.Hq / P.Hkv; P.n_seg = p->n_segments;
  P.r = r; P.g = g; P.n_sub = n_sub;
  for (int s = 0; s <= p->n_segments; ++s) P.seg_bounds[s] = p->seg_bounds[s];
  for (int i = 0; i <= n_sub; ++i) P.sub_bounds[i] = sub_bounds[i];
  P.Q = reinterpret_cast<const __nv_bfloat16*>(Q); P.K = reinterpret_cast<const __nv_bfloat16*>(K);
  P.rows = rows; P.A = A; P.lse = lse; P.colmass = colmass; P.diagmass = diagmass; P.descr = descr; P.rowstat = scratch;
  P.scale = (float)(1.0 / sqrt((double)RS_HEAD_DIM));
  const int nbg = P.n / g;
  // enough CTAs per KV head to fill the machine, at least kKB key blocks each
  int ctas = (2 * 148 + P.n_seg * P.Hkv - 1) / (P.n_seg * P.Hkv);
  int per = (nbg + ctas - 1) / ctas;
  per = (per + kKB - 1) / kKB * kKB;
  ctas = (nbg + per - 1) / per;
  const size_t smem = 128 * 256 * 2 + kKB * 128 * 4;
  static rs_smem_attr logits_attr;
  if (rs_ensure_dynamic_smem(logits_attr, rs_pp_logits_kernel, (int)smem) != RS_OK) return RS_ERR_CUDA;
  rs_pp_logits_kernel<<<dim3(ctas, P.n_seg * P.Hkv), 256, smem, stream>>>(P, per);
  rs_pp_softmax_kernel<<<dim3(r, P.n_seg * P.Hq), 256, 0, stream>>>(P);
  rs_pp_reduce_kernel<<<dim3((nbg + 255) / 256, P.n_seg * P.Hq), 256, 0, stream>>>(P);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
