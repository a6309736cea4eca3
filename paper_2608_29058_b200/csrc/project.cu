// The producer of Q, K, V: one layer's QKV projection with rotary position embedding on the tensor cores, with the
// side outputs of the attention probe leaving the same epilogue (Section 3.4: routing "runs ... concurrently with
// projection kernels or as a fused GPU reduction"; Section 3.1: "pooled queries and keys score coarse blocks";
// Eq. 5 needs max_j ||v_j||).
//
//   Y = X W^T      X [n, d_model] bf16, W [(Hq + 2 Hkv) * 128, d_model] bf16 (heads in the order Q.., K.., V..)
//   Q, K: rotate-half rotary embedding with cos / sin tables [n, 64]; V: as is.  Outputs bf16 [heads][n][128].
//   side outputs, from the ROUNDED bf16 values (what the probe would read back):
//     qpool [Hq][n/64][128], kpool [Hkv][n/64][128]   64-row means (fp32)
//     vbmax [Hkv][n/64]                               max over the block's rows of ||v||^2 (fp32)
//
// Persistent kernel, one CTA per SM.  A tile is 128 tokens x 256 output features (two heads): the TMA warp streams
// 128 x 64 slices of X and 256 x 64 slices of W through a four-stage ring (128-byte swizzle), the MMA warp issues
// tcgen05.mma M128 N256 K16 into one of two 256-column accumulators in TMEM, and four epilogue warps (one token per
// thread) rotate, round, store and reduce the tile that just finished while the next one is being multiplied.
#include "common.cuh"

namespace {

constexpr int kPjThreads = 192;          // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kPjStages = 4;
constexpr int kPjTileM = 128, kPjTileN = 256, kPjTileK = 64;
constexpr uint32_t kPjStageBytes = (kPjTileM + kPjTileN) * kPjTileK * 2;     // 48 KB
constexpr uint32_t kPjTmemCols = 512;

struct PjParams {
  int n, dm, Hq, Hkv;
  int m_tiles, n_tiles, k_blocks;
  const float* cos; const float* sin;     // [n][64]
  __nv_bfloat16 *Q, *K, *V;
  float *qpool, *kpool, *vbmax;            // each may be NULL
  int32_t* status;
};

struct PjSmem {
  static constexpr uint32_t stages = 0;                                   // kPjStages x (A 16 KB | B 32 KB)
  static constexpr uint32_t part = kPjStages * kPjStageBytes;            // [2][4 warps][256] fp32 column sums
  static constexpr uint32_t vmx = part + 2 * 4 * 256 * 4;                // [2][4 warps][2] fp32
  static constexpr uint32_t bars = vmx + 64;
  static constexpr uint32_t misc = bars + 128;
  static constexpr uint32_t total = misc + 64 + 1024;
};

// Sums v[0..31] over the 32 lanes of the warp; lane l ends with the sum of element l in v[0].  Fixed order.
__device__ __forceinline__ float warp_column_sums(float (&v)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < off; ++k) {
      const float send = up ? v[k] : v[k + off];
      const float recv = __shfl_xor_sync(0xffffffffu, send, off);
      v[k] = (up ? v[k + off] : v[k]) + recv;
    }
  }
  return v[0];
}

__global__ void __launch_bounds__(kPjThreads, 1)
rs_qkv_rope_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ PjParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + PjSmem::bars);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + PjSmem::misc);
  volatile int* abort_flag = misc + 1;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[4]);       // one per stage
  const uint32_t bar_tfull = smem_u32(&bars[8]), bar_tempty = smem_u32(&bars[10]);    // one per accumulator
  const uint32_t bar_epi = smem_u32(&bars[12]);                                        // the epilogue warps' own meeting point

  if (tid == 0) {
    for (uint32_t i = 0; i < kPjStages; ++i) { mbar_init(bar_full + 8u * i, 1); mbar_init(bar_empty + 8u * i, 1); }
    for (uint32_t i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8u * i, 1); mbar_init(bar_tempty + 8u * i, 4); }
    mbar_init(bar_epi, 128);
    misc[1] = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW);
  }
  if (warp == 1) { tmem_alloc(smem_u32((const void*)&misc[0]), kPjTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  const int n_tiles_total = P.m_tiles * P.n_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      bool ok = true;
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x) {
        const int mt = t / P.n_tiles, nt = t - mt * P.n_tiles;
        for (int kb = 0; kb < P.k_blocks; ++kb, ++it) {
          const uint32_t st = it % kPjStages, ph = (it / kPjStages) & 1u;
          ok = mbar_wait(bar_empty + 8u * st, ph ^ 1u, abort_flag);
          if (!ok) break;
          const uint32_t dst = base + PjSmem::stages + st * kPjStageBytes;
          mbar_arrive_expect_tx(bar_full + 8u * st, kPjStageBytes);
          tma_load_2d(dst, &tmX, bar_full + 8u * st, kb * kPjTileK, mt * kPjTileM);
          tma_load_2d(dst + kPjTileM * kPjTileK * 2, &tmW, bar_full + 8u * st, kb * kPjTileK, nt * kPjTileN);
        }
      }
      if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, 71); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      constexpr uint32_t idesc = umma_idesc_bf16(kPjTileM, kPjTileN, 0, 0);
      bool ok = true;
      int site = 72;
      uint32_t it = 0, tile_no = 0;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++tile_no) {
        const uint32_t acc = tile_no & 1u, aph = (tile_no >> 1) & 1u;
        ok = mbar_wait(bar_tempty + 8u * acc, aph ^ 1u, abort_flag); site = 72;
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + acc * 256u;
        for (int kb = 0; kb < P.k_blocks; ++kb, ++it) {
          const uint32_t st = it % kPjStages, ph = (it / kPjStages) & 1u;
          ok = mbar_wait(bar_full + 8u * st, ph, abort_flag); site = 73;
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_sm = base + PjSmem::stages + st * kPjStageBytes;
          const uint64_t adesc = umma_smem_desc(a_sm, 16, 1024);
          const uint64_t bdesc = umma_smem_desc(a_sm + kPjTileM * kPjTileK * 2, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)     // 16 elements of the reduction = 32 bytes along the swizzled row
            umma_ss(d_tmem, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), idesc, (kb | kk) != 0 ? 1u : 0u);
          umma_commit(bar_empty + 8u * st);
        }
        if (!ok) break;
        umma_commit(bar_tfull + 8u * acc);
      }
      if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, site); *abort_flag = 1; }
    }
  } else {
    // -------------------------------------------------------------------- epilogue: one token per thread
    const int ew = warp - 2;                   // 0..3
    const int quad = warp & 3;                 // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;            // row of the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    float* part = reinterpret_cast<float*>(sm + PjSmem::part);
    float* vmx = reinterpret_cast<float*>(sm + PjSmem::vmx);
    const int et = tid - 64;                   // 0..127
    bool ok = true;
    uint32_t tile_no = 0;
    for (int t = blockIdx.x; t < n_tiles_total; t += gridDim.x, ++tile_no) {
      const int mt = t / P.n_tiles, nt = t - mt * P.n_tiles;
      const uint32_t acc = tile_no & 1u, aph = (tile_no >> 1) & 1u, par = tile_no & 1u;
      ok = mbar_wait(bar_tfull + 8u * acc, aph, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const int tok = mt * kPjTileM + r;
      const bool valid = tok < P.n;
      const int tok_c = valid ? tok : 0;
      float* my_part = part + (par * 4 + quad) * 256;
#pragma unroll 1
      for (int hh = 0; hh < 2; ++hh) {
        const int H = nt * 2 + hh;             // head in the order Q.., K.., V..
        const bool is_v = H >= P.Hq + P.Hkv;
        __nv_bfloat16* dst;
        if (H < P.Hq) dst = P.Q + ((size_t)H * P.n + tok_c) * RS_HEAD_DIM;
        else if (!is_v) dst = P.K + ((size_t)(H - P.Hq) * P.n + tok_c) * RS_HEAD_DIM;
        else dst = P.V + ((size_t)(H - P.Hq - P.Hkv) * P.n + tok_c) * RS_HEAD_DIM;
        float sq = 0.f;
#pragma unroll 1
        for (int c = 0; c < 64; c += 32) {     // dimensions [c, c + 32) and their partners [64 + c, 64 + c + 32)
          uint32_t lo[32], hi[32];
          tmem_ld32(tmem + lane_addr + acc * 256u + (uint32_t)(hh * 128 + c), lo);
          tmem_ld32(tmem + lane_addr + acc * 256u + (uint32_t)(hh * 128 + 64 + c), hi);
          tc_wait_ld();
          float a[32], b[32];
          if (!is_v) {
            const float4* c4 = reinterpret_cast<const float4*>(P.cos + (size_t)tok_c * 64 + c);
            const float4* s4 = reinterpret_cast<const float4*>(P.sin + (size_t)tok_c * 64 + c);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 cc = __ldg(c4 + q), ss = __ldg(s4 + q);
              const float cv[4] = {cc.x, cc.y, cc.z, cc.w}, sv[4] = {ss.x, ss.y, ss.z, ss.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float x0 = __uint_as_float(lo[4 * q + e]), x1 = __uint_as_float(hi[4 * q + e]);
                a[4 * q + e] = x0 * cv[e] - x1 * sv[e];
                b[4 * q + e] = x1 * cv[e] + x0 * sv[e];
              }
            }
          } else {
#pragma unroll
            for (int q = 0; q < 32; ++q) { a[q] = __uint_as_float(lo[q]); b[q] = __uint_as_float(hi[q]); }
          }
          // round once to bf16; the side outputs are formed from the rounded values
          uint32_t pa[16], pb[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            pa[q] = pack_bf16x2(a[2 * q], a[2 * q + 1]);
            pb[q] = pack_bf16x2(b[2 * q], b[2 * q + 1]);
            a[2 * q] = __uint_as_float(pa[q] << 16); a[2 * q + 1] = __uint_as_float(pa[q] & 0xffff0000u);
            b[2 * q] = __uint_as_float(pb[q] << 16); b[2 * q + 1] = __uint_as_float(pb[q] & 0xffff0000u);
          }
          if (valid) {
            uint4* d0 = reinterpret_cast<uint4*>(dst + c);
            uint4* d1 = reinterpret_cast<uint4*>(dst + 64 + c);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              d0[q] = make_uint4(pa[4 * q], pa[4 * q + 1], pa[4 * q + 2], pa[4 * q + 3]);
              d1[q] = make_uint4(pb[4 * q], pb[4 * q + 1], pb[4 * q + 2], pb[4 * q + 3]);
            }
          }
          if (is_v) {
#pragma unroll
            for (int q = 0; q < 32; ++q) { sq = fmaf(a[q], a[q], sq); sq = fmaf(b[q], b[q], sq); }
          } else {
            if (!valid) {
#pragma unroll
              for (int q = 0; q < 32; ++q) { a[q] = 0.f; b[q] = 0.f; }
            }
            const float sa = warp_column_sums(a, lane), sb = warp_column_sums(b, lane);
            my_part[hh * 128 + c + lane] = sa;
            my_part[hh * 128 + 64 + c + lane] = sb;
          }
        }
        if (is_v) {
          float mx = valid ? sq : 0.f;
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
          if (lane == 0) vmx[(par * 4 + quad) * 2 + hh] = mx;
        }
      }
      // the accumulator is free again: the tensor cores may start the tile after next
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * acc);
      // the four warps meet, then every thread folds two warps' partial sums of two columns
      mbar_arrive(bar_epi);
      ok = mbar_wait(bar_epi, tile_no & 1u, abort_flag);
      if (!ok) break;
      const int blk0 = mt * 2;                 // first 64-token block of the tile
      for (int col = et; col < 512; col += 128) {          // (block b, head hh, dimension)
        const int b = col >> 8, hh = (col >> 7) & 1, dim = col & 127;
        const int H = nt * 2 + hh, blk = blk0 + b;
        if (blk * 64 >= P.n) continue;
        float* out = nullptr;
        if (H < P.Hq) out = P.qpool ? P.qpool + ((size_t)H * (P.n >> 6) + blk) * RS_HEAD_DIM : nullptr;
        else if (H < P.Hq + P.Hkv) out = P.kpool ? P.kpool + ((size_t)(H - P.Hq) * (P.n >> 6) + blk) * RS_HEAD_DIM : nullptr;
        if (out != nullptr) {
          // quadrants 0, 1 hold rows 0..63, quadrants 2, 3 rows 64..127 (the epilogue warps' quadrants are warp % 4)
          const float s0 = part[(par * 4 + 2 * b) * 256 + hh * 128 + dim], s1 = part[(par * 4 + 2 * b + 1) * 256 + hh * 128 + dim];
          out[dim] = (s0 + s1) * (1.0f / 64.0f);
        }
      }
      if (et < 4 && P.vbmax != nullptr) {
        const int b = et >> 1, hh = et & 1;
        const int H = nt * 2 + hh, blk = blk0 + b;
        if (H >= P.Hq + P.Hkv && blk * 64 < P.n)
          P.vbmax[(size_t)(H - P.Hq - P.Hkv) * (P.n >> 6) + blk] =
              fmaxf(vmx[(par * 4 + 2 * b) * 2 + hh], vmx[(par * 4 + 2 * b + 1) * 2 + hh]);
      }
    }
    if (!ok && lane == 0 && ew == 0) { rs_report(P.status, RS_ERR_TIMEOUT, 74); *abort_flag = 1; }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, kPjTmemCols); }
}

// vmax[s][g] = sqrt(max over the key blocks below the end of segment s of the block maxima of ||v||^2)
struct SegEnds { int v[RS_MAX_SEGMENTS]; };
__global__ void rs_pj_vmax_kernel(int Hkv, int nb, SegEnds ends, const float* vbmax, float* vmax) {
  const int s = blockIdx.x / Hkv, g = blockIdx.x % Hkv;
  const int nbs = ends.v[s];
  float m = 0.f;
  for (int i = threadIdx.x; i < nbs; i += blockDim.x) m = fmaxf(m, vbmax[(size_t)g * nb + i]);
  __shared__ float red[32];
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < (int)(blockDim.x >> 5); ++i) m = fmaxf(m, red[i]);
    vmax[blockIdx.x] = sqrtf(m);
  }
}

}  // namespace

extern "C" int rs_qkv_rope_project(int n_tokens, int d_model, int n_q_heads, int n_kv_heads, const void* X, const void* W,
                                   const float* rope_cos, const float* rope_sin, void* Q, void* K, void* V, float* qpool,
                                   float* kpool, float* vbmax, int32_t* status, void* stream_) {
  if (n_tokens <= 0 || n_tokens % RS_BLOCK != 0 || d_model <= 0 || d_model % kPjTileK != 0) return RS_ERR_UNSUPPORTED_SHAPE;
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0) return RS_ERR_INVALID_ARG;
  if ((n_q_heads & 1) || (n_kv_heads & 1)) return RS_ERR_UNSUPPORTED_SHAPE;       // a tile holds two heads of one kind
  if (!X || !W || !rope_cos || !rope_sin || !Q || !K || !V) return RS_ERR_INVALID_ARG;
  if ((long long)n_q_heads * n_tokens >= (1ll << 31)) return RS_ERR_UNSUPPORTED_SHAPE;
  int rc = rs_check_device();
  if (rc != RS_OK) return rc;
  PjParams P{};
  P.n = n_tokens; P.dm = d_model; P.Hq = n_q_heads; P.Hkv = n_kv_heads;
  P.m_tiles = (n_tokens + kPjTileM - 1) / kPjTileM;
  P.n_tiles = (n_q_heads + 2 * n_kv_heads) * RS_HEAD_DIM / kPjTileN;
  P.k_blocks = d_model / kPjTileK;
  P.cos = rope_cos; P.sin = rope_sin;
  P.Q = reinterpret_cast<__nv_bfloat16*>(Q); P.K = reinterpret_cast<__nv_bfloat16*>(K); P.V = reinterpret_cast<__nv_bfloat16*>(V);
  P.qpool = qpool; P.kpool = kpool; P.vbmax = vbmax; P.status = status;
  CUtensorMap tmX, tmW;
  if (rs_make_tmap_bf16_2d(&tmX, X, (uint64_t)n_tokens, (uint64_t)d_model, kPjTileM, kPjTileK) ||
      rs_make_tmap_bf16_2d(&tmW, W, (uint64_t)(n_q_heads + 2 * n_kv_heads) * RS_HEAD_DIM, (uint64_t)d_model, kPjTileN, kPjTileK))
    return RS_ERR_CUDA;
  static rs_smem_attr attr;
  if (rs_ensure_dynamic_smem(attr, rs_qkv_rope_kernel, (int)PjSmem::total) != RS_OK) return RS_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return RS_ERR_CUDA;
  const int tiles = P.m_tiles * P.n_tiles;
  const int grid = tiles < sms ? tiles : sms;
  rs_qkv_rope_kernel<<<grid, kPjThreads, PjSmem::total, (cudaStream_t)stream_>>>(tmX, tmW, P);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

extern "C" int rs_value_norm_max(const rs_problem* p, const float* vbmax, float* vmax, int32_t* status, void* stream_) {
  (void)status;
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!vbmax || !vmax) return RS_ERR_INVALID_ARG;
  SegEnds ends{};
  for (int s = 0; s < p->n_segments; ++s) ends.v[s] = p->seg_bounds[s + 1] / RS_BLOCK;
  rs_pj_vmax_kernel<<<p->n_segments * p->n_kv_heads, 256, 0, (cudaStream_t)stream_>>>(p->n_kv_heads, p->n_keys / RS_BLOCK,
                                                                                      ends, vbmax, vmax);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
