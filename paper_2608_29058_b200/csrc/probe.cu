// Shared attention probe (Eq. 3, Section 3.2) in the last-64-query form, plus the pooled means for the
// coarse block scores and the value norms of Eq. 5.
//
// For every (segment, KV head) the 64 probe rows of up to four query heads (256 rows) are scored against all
// causal keys on the tensor cores, twice:
//   pass 1 (probe_lse):   S = Qp K^T with probe rows on the TMEM lanes; a thread owns one probe row and half of the
//                         tile's key columns and keeps a running maximum and sum; the partials of all key ranges are
//                         merged in the prologue of pass 2.  Two more warps form the 64-row means of K from the very
//                         tile the tensor cores read (no second stream of K for the pooled keys).
//   pass 2 (probe_accum): S^T = K Qp^T with keys on the TMEM lanes; every thread owns one key, so the column
//                         mass of a 16-row probe group is a sum inside the thread; the diagonal (slash) mass is a
//                         skewed sum over the warp's own 16 x 32 probabilities, formed by rotating every row over
//                         the lanes.  The four lane quadrants of a tile hold four different stretches of the CTA's
//                         key range (four TMA boxes of 32 keys), so a warp walks 32 consecutive keys per step through
//                         a contiguous quarter of the range and the part of a diagonal that runs off its 32 keys is
//                         carried, in a register, into its own next step.  Every offset is produced by exactly one
//                         thread: no atomics, no zero-filled output, no barrier between warps.  The same pass turns
//                         the block maxima of ||v||^2 into V_max and pools the last query block of every segment.
// Each key tile is read from HBM once per pass (TMA, 128-byte swizzle).
#include <type_traits>

#include "common.cuh"

namespace {

constexpr int RS_LOCAL_BAND = 1024;     // keys with i - j below this count as the row's local band
constexpr int kHC = 4;                 // head slots per CTA (4 x 64 = 256 probe rows)
constexpr int kRows = kHC * RS_PROBE_ROWS;
constexpr int kKeyTile = 128;
constexpr int kStages1 = 5;            // K-tile ring of pass 1
constexpr int kStages2 = 5;            // K-tile ring of pass 2
constexpr int kThreads1 = 640;         // pass 1: warp 0 TMA, warp 1 MMA, warps 2..17 compute, warps 18..19 pool K
constexpr int kThreads2 = 576;         // pass 2: warp 0 TMA, warp 1 MMA, warps 2..17 compute
constexpr int kComputeThreads = 512;
constexpr uint32_t kTmemCols = 512;

struct rs_candidate_list { int32_t pattern[RS_MAX_CANDIDATES]; };

struct ProbeParams {
  int n, Hq, Hkv, group, n_seg, n_hc;  // n_hc = head chunks per KV head = ceil(group / 4)
  int seg_bounds[RS_MAX_SEGMENTS + 1];
  int run_start[RS_MAX_SEGMENTS][RS_PROBE_GROUPS];   // first row of each 16-row group of probe rows, per segment
  int n_splits, per;
  float4* partial;    // [n_seg*Hkv*n_hc][2*n_splits][256] (max, sum, sum of p * score, sum of p inside the local band), exp2 domain
  float* lse_probe;   // [Hq][n_seg][64]
  float* descr;       // [n_seg][Hq][2] entropy and local-band mass, means over the 64 probe rows (may be NULL)
  float* vert;        // [n_seg][Hq][4][n]
  float* slash;       // [n_seg][Hq][4][n]
  float* kpool;       // [Hkv][n/64][128] 64-row means of K, written by pass 1 (may be NULL)
  const float* blockmax;  // [Hkv][n/64] block maxima of ||v||^2, complete before pass 2 starts (may be NULL)
  float* vmax;        // [n_seg][Hkv] written by pass 2 from blockmax (may be NULL)
  float* qpool_last;  // [Hq][n/64][128]: pass 2 writes the mean of every segment's last 64 query rows (may be NULL)
  int32_t* status;
  float scale_log2e;
};

template <int PASS>
struct SmemT {
  static constexpr int stages = PASS == 1 ? kStages1 : kStages2;
  static constexpr uint32_t qp = 0;                       // 2 halves x 256 rows x 128 B
  static constexpr uint32_t k = 65536;                    // stages x (2 halves x 128 rows x 128 B)
  static constexpr uint32_t x = k;                        // pass 2: scratch of the prologue (the ring is not yet in use)
  static constexpr uint32_t lse = k + stages * 32768;     // 256 floats
  static constexpr uint32_t bars = lse + 1024;            // mbarriers
  static constexpr uint32_t misc = bars + 256;
  static constexpr uint32_t total = misc + 64 + 1024;     // + alignment slack
};
static_assert(SmemT<1>::total <= 227 * 1024 && SmemT<2>::total <= 227 * 1024, "probe shared memory");

__device__ __forceinline__ float max3f(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

template <int PASS>
__global__ void __launch_bounds__(PASS == 1 ? kThreads1 : kThreads2, 1)
rs_probe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ ProbeParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int kThreads = PASS == 1 ? kThreads1 : kThreads2;
  using Smem = SmemT<PASS>;
  constexpr int kStages = Smem::stages;

  // unit = (segment, kv head, head chunk); blockIdx.x = split of the key range
  const int unit = blockIdx.y;
  const int hc = unit % P.n_hc;
  const int g = (unit / P.n_hc) % P.Hkv;
  const int s = unit / (P.n_hc * P.Hkv);
  const int q1 = P.seg_bounds[s + 1];
  const int h0 = g * P.group + hc * kHC;
  const int n_heads = min(kHC, P.group - hc * kHC);
  const int n_tiles = (q1 + kKeyTile - 1) / kKeyTile;
  const int per = P.per;                      // key tiles per CTA, the same for every unit
  const int t0 = blockIdx.x * per, t1 = min(n_tiles, t0 + per);
  int run0[RS_PROBE_GROUPS];               // first row of each group of probe rows
#pragma unroll
  for (int q = 0; q < RS_PROBE_GROUPS; ++q) run0[q] = P.run_start[s][q];
  const int i_min = min(min(run0[0], run0[1]), min(run0[2], run0[3]));   // lowest probe row
  // Pass 2: the CTA's keys [128 t0, 128 t1) are cut into four contiguous quarters of 32 (t1 - t0) keys, one per lane
  // quadrant; step st = -1 .. t1 - t0 - 1 of quadrant q covers keys quarter start + 32 st .. + 31.  Step -1 stores
  // nothing: it only produces the carries of the diagonals that reach back over the start of the quarter.
  const int n_mma = (PASS == 2) ? (t1 - t0 + 1) : (t1 - t0);      // tiles through the tensor cores
  // pass 1: the CTAs of the last segment (it sees every key) and of the first head chunk also pool K
  const bool do_pool = PASS == 1 && P.kpool != nullptr && s == P.n_seg - 1 && hc == 0;

  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + Smem::bars);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + Smem::misc);
  volatile int* abort_flag = misc + 1;
  float* s_lse = reinterpret_cast<float*>(sm + Smem::lse);
  const uint32_t bar_q = smem_u32(&bars[0]);
  uint32_t bar_full[kStages], bar_empty[kStages], bar_tfull[2], bar_tempty[2];
#pragma unroll
  for (int i = 0; i < kStages; ++i) { bar_full[i] = smem_u32(&bars[1 + i]); bar_empty[i] = smem_u32(&bars[1 + kStages + i]); }
#pragma unroll
  for (int i = 0; i < 2; ++i) { bar_tfull[i] = smem_u32(&bars[1 + 2 * kStages + i]); bar_tempty[i] = smem_u32(&bars[3 + 2 * kStages + i]); }

  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int i = 0; i < kStages; ++i) { mbar_init(bar_full[i], 1); mbar_init(bar_empty[i], do_pool ? 3 : 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull[i], 1); mbar_init(bar_tempty[i], kComputeThreads / 32); }
    misc[1] = 0;
    misc[2] = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK);
  }
  if (warp == 1) { tmem_alloc(smem_u32((const void*)&misc[0]), kTmemCols); tmem_relinquish(); }
  if (PASS == 2) {
    // Merge of pass 1's partial (max, sum) pairs into the log-sum-exp of the unit's 256 probe rows; every CTA of the
    // unit forms the same values in the same order, the first one also stores them (and the two descriptors).
    // 512 threads: thread (row, half) folds every second partial of the row, eight loads in flight at a time; the two
    // halves meet through shared memory.  The order of the additions is fixed, so every CTA gets the same bits.
    float4* mrg = reinterpret_cast<float4*>(sm + Smem::x);        // [2][256] (max, sum, a, loc)
    const int n_part = 2 * P.n_splits;
    if (tid < 2 * kRows) {
      const int row = tid & (kRows - 1), half = tid >> 8;
      const float4* part = P.partial + (size_t)unit * n_part * kRows + row;
      float m = -INFINITY, l = 0.f, a = 0.f, loc = 0.f;
      for (int k0 = half; k0 < n_part; k0 += 16) {
        float4 pk[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int k = k0 + 2 * u;
          pk[u] = k < n_part ? __ldg(part + (size_t)k * kRows) : make_float4(-INFINITY, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (pk[u].x > m) {
            const float sc = exp2f(m - pk[u].x);
            l *= sc; a *= sc; loc *= sc;
            m = pk[u].x;
          }
          if (pk[u].x > -INFINITY) {
            const float sc = exp2f(pk[u].x - m);
            l = fmaf(pk[u].y, sc, l); a = fmaf(pk[u].z, sc, a); loc = fmaf(pk[u].w, sc, loc);
          }
        }
      }
      mrg[half * kRows + row] = make_float4(m, l, a, loc);
    }
    __syncthreads();
    if (tid < kRows) {
      const int row = tid, hh = row >> 6;
      const float4 p0 = mrg[row], p1 = mrg[kRows + row];
      const float m = fmaxf(p0.x, p1.x);
      const float s0 = p0.x > -INFINITY ? exp2f(p0.x - m) : 0.f, s1 = p1.x > -INFINITY ? exp2f(p1.x - m) : 0.f;
      const float l = p0.y * s0 + p1.y * s1, a = p0.z * s0 + p1.z * s1, loc = p0.w * s0 + p1.w * s1;
      const float lse2 = m + log2f(l);
      s_lse[row] = lse2;
      const bool live = hh < n_heads;
      if (blockIdx.x == 0 && live)
        P.lse_probe[((size_t)(h0 + hh) * P.n_seg + s) * RS_PROBE_ROWS + (row & 63)] = lse2 * 0.6931471805599453f;
      if (blockIdx.x == 0 && P.descr != nullptr) {
        // H_i = -sum p ln p = ln 2 * (lse2 - E_p[score2]); local mass = local sum / l; then the mean over the head's
        // 64 rows (fixed order: a butterfly inside each warp, then the two warps of a head)
        float e = 0.6931471805599453f * (lse2 - a / l), lc = loc / l;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          e += __shfl_xor_sync(0xffffffffu, e, off);
          lc += __shfl_xor_sync(0xffffffffu, lc, off);
        }
        float* red = reinterpret_cast<float*>(sm + Smem::x) + 4 * 2 * kRows;      // behind the merge scratch
        if (lane == 0) { red[2 * warp] = e; red[2 * warp + 1] = lc; }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (PASS == 2 && blockIdx.x == 0 && P.descr != nullptr && tid < n_heads) {
    const float* red = reinterpret_cast<const float*>(sm + Smem::x) + 4 * 2 * kRows;
    const int h = h0 + tid;
    P.descr[((size_t)s * P.Hq + h) * 2 + 0] = (red[4 * tid] + red[4 * tid + 2]) * (1.0f / 64.0f);
    P.descr[((size_t)s * P.Hq + h) * 2 + 1] = (red[4 * tid + 1] + red[4 * tid + 3]) * (1.0f / 64.0f);
  }
  // pass 2's scratch lies in the first stage of the ring: its generic-proxy accesses are ordered before the TMA writes
  if (PASS == 2) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  const uint32_t tmem = (uint32_t)misc[0];
  if (t0 >= t1) {   // nothing to do for this split (uniform across the CTA)
    if (PASS == 1) {
      for (int i = tid; i < 2 * kRows; i += kThreads)
        P.partial[((size_t)unit * 2 * P.n_splits + 2 * blockIdx.x) * kRows + i] = make_float4(-INFINITY, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    return;
  }

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- producer
      mbar_arrive_expect_tx(bar_q, (uint32_t)n_heads * 16384u);
      for (int hh = 0; hh < n_heads; ++hh) {
#pragma unroll
        for (int q = 0; q < RS_PROBE_GROUPS; ++q) {      // one box of 16 rows per group
          const int row = (h0 + hh) * P.n + run0[q];
          tma_load_2d(base + Smem::qp + (uint32_t)hh * 8192u + (uint32_t)q * 2048u, &tmQ, bar_q, 0, row);
          tma_load_2d(base + Smem::qp + 32768u + (uint32_t)hh * 8192u + (uint32_t)q * 2048u, &tmQ, bar_q, 64, row);
        }
      }
      bool ok = true;
      for (int it = 0; it < n_mma; ++it) {
        const int st = it % kStages;
        ok = mbar_wait(bar_empty[st], ((uint32_t)(it / kStages) & 1u) ^ 1u, abort_flag);
        if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, 11); break; }
        mbar_arrive_expect_tx(bar_full[st], 32768u);
        const uint32_t dst = base + Smem::k + (uint32_t)st * 32768u;
        if (PASS == 1) {
          const int row = g * P.n + (t0 + it) * kKeyTile;
          tma_load_2d(dst, &tmK, bar_full[st], 0, row);
          tma_load_2d(dst + 16384u, &tmK, bar_full[st], 64, row);
        } else {
          // rows 32 q .. 32 q + 31 of the tile = the 32 keys of quadrant q's current step (a step that would start
          // before key 0 loads keys 0..31 instead; its probabilities are zeroed by the consumer)
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int key0 = max(0, t0 * kKeyTile + (q * (t1 - t0) + it - 1) * 32);
            tma_load_2d(dst + (uint32_t)q * 4096u, &tmK, bar_full[st], 0, g * P.n + key0);
            tma_load_2d(dst + 16384u + (uint32_t)q * 4096u, &tmK, bar_full[st], 64, g * P.n + key0);
          }
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (PASS == 2 && blockIdx.x == 0 && hc == 0 && P.vmax != nullptr) {
      // vmax[s][g] = sqrt(max over the key blocks below the segment end of the block maxima of ||v||^2), by the 31
      // lanes of this warp that have nothing else to do (a maximum does not depend on the order)
      const int nbs = q1 >> 6;
      const float* bm = P.blockmax + (size_t)g * (P.n >> 6);
      float m = 0.f;
      for (int i = lane - 1; i < nbs; i += 31) m = fmaxf(m, __ldg(bm + i));
      atomicMax(const_cast<int*>(&misc[2]), __float_as_int(m));      // non-negative floats order like their bit patterns
      __syncwarp(0xfffffffeu);
      if (lane == 1) P.vmax[s * P.Hkv + g] = sqrtf(__int_as_float(misc[2]));
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      int site = 12;
      for (int it = 0; it < n_mma && ok; ++it) {
        const int st = it % kStages, b = it & 1;
        ok = mbar_wait(bar_full[st], (uint32_t)(it / kStages) & 1u, abort_flag); site = 13;
        if (!ok) break;
        ok = mbar_wait(bar_tempty[b], ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag); site = 14;
        if (!ok) break;
        tc_fence_after();
        const uint32_t ksm = base + Smem::k + (uint32_t)st * 32768u;
        if (PASS == 1) {
          // probe rows on lanes: two M=128 products (head pairs), N = 128 keys
          const uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);
          for (int pr = 0; pr < 2; ++pr) {
            const uint64_t adesc = umma_smem_desc(base + Smem::qp + (uint32_t)pr * 16384u, 16, 1024);
            const uint64_t bdesc = umma_smem_desc(ksm, 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint64_t aoff = (uint64_t)(((kk >> 2) * 32768 + (kk & 3) * 32) >> 4);
              const uint64_t boff = (uint64_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
              umma_ss(tmem + (uint32_t)(b * 256 + pr * 128), adesc + aoff, bdesc + boff, idesc, kk > 0 ? 1u : 0u);
            }
          }
        } else {
          // keys on lanes: one M=128 product, N = 256 probe rows
          const uint32_t idesc = umma_idesc_bf16(128, 256, 0, 0);
          const uint64_t adesc = umma_smem_desc(ksm, 16, 1024);
          const uint64_t bdesc = umma_smem_desc(base + Smem::qp, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t aoff = (uint64_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
            const uint64_t boff = (uint64_t)(((kk >> 2) * 32768 + (kk & 3) * 32) >> 4);
            umma_ss(tmem + (uint32_t)(b * 256), adesc + aoff, bdesc + boff, idesc, kk > 0 ? 1u : 0u);
          }
        }
        umma_commit(bar_tfull[b]);
        umma_commit(bar_empty[st]);
      }
      if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, site); *abort_flag = 1; }
    }
  } else if (PASS == 1 && warp >= 18) {
    // ------------------------------------------------------------------ 64-row means of K from the staged tiles
    if (do_pool) {
      const int w = warp - 18;                  // key block inside the tile
      const int c = lane & 15, par = lane >> 4; // 16-byte column chunk, row parity
      const uint32_t col_off = (uint32_t)(c >> 3) * 16384u;
      const int cc = c & 7;
      bool ok = true;
      for (int t = t0; t < t1; ++t) {
        const int it = t - t0, st = it % kStages;
        ok = mbar_wait(bar_full[st], (uint32_t)(it / kStages) & 1u, abort_flag);
        if (!ok) break;
        const int kb = 2 * t + w;
        if (kb * 64 < q1) {
          const uint8_t* tile = sm + Smem::k + (uint32_t)st * 32768u + col_off;
          float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll 8
          for (int k = 0; k < 32; ++k) {
            const int r = 64 * w + 2 * k + par;
            const uint4 u = *reinterpret_cast<const uint4*>(tile + r * 128 + ((cc ^ (r & 7)) << 4));   // 128-byte swizzle
            const uint32_t wd[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              acc[2 * e] += __uint_as_float(wd[e] << 16);
              acc[2 * e + 1] += __uint_as_float(wd[e] & 0xffff0000u);
            }
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);
          if (par == 0) {
            float4* dst = reinterpret_cast<float4*>(P.kpool + ((size_t)g * (P.n >> 6) + kb) * RS_HEAD_DIM + c * 8);
            const float sc = 1.0f / 64.0f;
            dst[0] = make_float4(acc[0] * sc, acc[1] * sc, acc[2] * sc, acc[3] * sc);
            dst[1] = make_float4(acc[4] * sc, acc[5] * sc, acc[6] * sc, acc[7] * sc);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty[st]);
      }
      if (!ok && lane == 0) { rs_report(P.status, RS_ERR_TIMEOUT, 16); *abort_flag = 1; }
    }
  } else {
    // ------------------------------------------------------------------ compute warps
    const int cw = warp - 2;                 // 0..15
    const int quad = warp & 3;               // TMEM lane quadrant this warp may touch
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const float sl2 = P.scale_log2e;
    bool ok = true;

    if (PASS == 2 && blockIdx.x == 0 && P.qpool_last != nullptr) {
      // 64-row mean of the segment's last query block from the staged probe rows (the same rows).  One thread per
      // (head slot, dimension); the additions run in the order of the streaming pool kernel (rows r, r + 16, r + 32,
      // r + 48 first, then r = 0 .. 15), so both give the same bits.
      ok = mbar_wait(bar_q, 0, abort_flag);
      const int ct = tid - 64, hh = ct >> 7, x = ct & 127;
      if (ok && hh < n_heads) {
        const uint8_t* qh = sm + Smem::qp + (uint32_t)(x >> 6) * 32768u + (uint32_t)hh * 8192u + (uint32_t)(x & 7) * 2u;
        const int chunk = (x & 63) >> 3;
        float sum = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          float acc = 0.f;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint16_t u = *reinterpret_cast<const uint16_t*>(qh + k * 2048 + r * 128 + ((chunk ^ (r & 7)) << 4));
            acc += __uint_as_float((uint32_t)u << 16);
          }
          sum += acc;
        }
        P.qpool_last[((size_t)(h0 + hh) * (P.n >> 6) + ((q1 >> 6) - 1)) * RS_HEAD_DIM + x] = sum * (1.0f / 64.0f);
      }
    }

    if (PASS == 1) {
      const int part = (cw >> 2) & 1;                 // head pair
      const int colhalf = cw >> 3;                    // which 64 of the tile's 128 key columns
      const int r = quad * 32 + lane;                 // row inside the head pair (0..127)
      const int hh = part * 2 + (r >> 6);             // head slot
      const int i = run0[(r & 63) >> 4] + (r & 15);   // global query row
      const bool want_descr = P.descr != nullptr;
      float m_run = -INFINITY, l_run = 0.f;
      float a_run = 0.f, loc_run = 0.f;               // sum of p * score and local-band sum of p (descriptors)
      uint32_t v[32];
      for (int t = t0; t < t1; ++t) {
        const int it = t - t0, b = it & 1;
        ok = mbar_wait(bar_tfull[b], (uint32_t)(it >> 1) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const int j0 = t * kKeyTile + colhalf * 64;
        const bool need_mask = j0 + 63 > i_min;
        const bool near = j0 + 63 > i_min - RS_LOCAL_BAND;   // may reach into some row's local band
#pragma unroll 1
        for (int c2 = 0; c2 < 2; ++c2) {
          tmem_ld32(tmem + lane_addr + (uint32_t)(b * 256 + part * 128 + colhalf * 64 + c2 * 32), v);
          tc_wait_ld();
          const int jc = j0 + c2 * 32;
          if (need_mask) {
#pragma unroll
            for (int x = 0; x < 32; ++x)
              if (jc + x > i) v[x] = 0xff800000u;
          }
          float mxa[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            mxa[q] = max3f(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1]), __uint_as_float(v[8 * q + 2]));
            mxa[q] = max3f(mxa[q], __uint_as_float(v[8 * q + 3]), __uint_as_float(v[8 * q + 4]));
            mxa[q] = max3f(mxa[q], __uint_as_float(v[8 * q + 5]), __uint_as_float(v[8 * q + 6]));
            mxa[q] = fmaxf(mxa[q], __uint_as_float(v[8 * q + 7]));
          }
          const float mx = fmaxf(max3f(mxa[0], mxa[1], mxa[2]), mxa[3]) * sl2;
          // the reference only moves when it is exceeded by more than 2^8 (the sums stay far inside fp32 range)
          if (mx > m_run + 8.0f) {
            const float sc = fast_exp2(m_run - mx);
            l_run *= sc; a_run *= sc; loc_run *= sc;
            m_run = mx;
          }
          if (m_run > -INFINITY) {
            const float neg_m = -m_run;
            if (want_descr) {
              float acc = 0.f, acc_a = 0.f, acc_l = 0.f;
#pragma unroll
              for (int x = 0; x < 32; ++x) {
                const float sv = __uint_as_float(v[x]) * sl2;
                const float pe = fast_exp2(sv + neg_m);
                acc += pe;
                acc_a = fmaf(pe, fmaxf(sv, -1e30f), acc_a);          // masked entries: pe = 0, keep the product finite
                if (near && i - (jc + x) < RS_LOCAL_BAND) acc_l += pe;
              }
              l_run += acc; a_run += acc_a; loc_run += acc_l;
            } else {
              float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int x = 0; x < 32; x += 4) {
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] += fast_exp2(fmaf(__uint_as_float(v[x + q]), sl2, neg_m));
              }
              l_run += (acc[0] + acc[1]) + (acc[2] + acc[3]);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty[b]);   // one arrival per warp: 512 arrivals per tile queue up on the barrier
      }
      if (ok) {
        P.partial[((size_t)unit * 2 * P.n_splits + 2 * blockIdx.x + colhalf) * kRows + hh * 64 + (r & 63)] =
            make_float4(m_run, l_run, a_run, loc_run);
      }
    } else {
      // Sixteen warps: warp (quad, hh) owns the 32 keys of its quadrant's current step (its TMEM lanes) and the 64
      // probe rows of head slot hh.  Per probe group: 16 probabilities per key, their sum is the column mass; the
      // diagonal mass is a skewed sum over the warp's 16 x 32 probabilities: lane l sums row r's entry of key
      // l - 15 + r, the diagonal that ends at its key in row 15 (offset o = first row of the group + 15 - key), fetched
      // by rotating every row over the lanes.  The terms of that diagonal that lie in the previous step's keys arrive
      // through a register: lanes 0..14 also sum the part of the diagonal ending at the same lane's key of the NEXT
      // step that lies in this step's keys (the wrapped-around end of the same rotations), and carry it over.
      const int hh = cw >> 2;                         // head slot
      const bool live = hh < n_heads;
      const int key_q = t0 * kKeyTile + quad * (t1 - t0) * 32;     // first key of this quadrant's quarter
      float carry[RS_PROBE_GROUPS] = {0.f, 0.f, 0.f, 0.f};
      float* const vert_h = P.vert + ((size_t)s * P.Hq + (size_t)(h0 + hh)) * RS_PROBE_GROUPS * (size_t)P.n;
      float* const slash_h = P.slash + ((size_t)s * P.Hq + (size_t)(h0 + hh)) * RS_PROBE_GROUPS * (size_t)P.n;
      // One step: the four probe groups of the warp's 32 keys.  MASKED steps (those that reach some probe row, and the
      // step before key 0) also zero the probabilities of pairs with j > i or j < 0, and skip a group altogether when
      // all of the step's keys lie behind the group's last row.  Every thread writes one column mass and one diagonal
      // mass per group: the diagonal that ends at its key, offset o = first row of the group + 15 - key, or, when that
      // is negative, the zero of the offset equal to its key (offsets beyond the group's reach have no key at all).
      auto step = [&](auto masked_tag, int b, int jw, bool store) {
        constexpr bool MASKED = decltype(masked_tag)::value;
        const int j = jw + lane;
        uint32_t v16[16];
        const uint32_t t_hh = tmem + lane_addr + (uint32_t)(b * 256 + hh * 64);
        tmem_ld16(t_hh, v16);
#pragma unroll
        for (int grp = 0; grp < RS_PROBE_GROUPS; ++grp) {
          const int ig = run0[grp];                     // first row of the group
          const float4* l4 = reinterpret_cast<const float4*>(s_lse + hh * 64 + grp * 16);
          float lse16[16];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float4 t4 = l4[q];
            lse16[4 * q] = t4.x; lse16[4 * q + 1] = t4.y; lse16[4 * q + 2] = t4.z; lse16[4 * q + 3] = t4.w;
          }
          tc_wait_ld16(v16);
          if (MASKED && jw > ig + 15) {                 // uniform over the warp: no key of the step is visible to the group
            if (grp + 1 < RS_PROBE_GROUPS) tmem_ld16(t_hh + (uint32_t)(grp + 1) * 16u, v16);
            if (store && j < q1) { vert_h[(size_t)grp * P.n + j] = 0.f; slash_h[(size_t)grp * P.n + j] = 0.f; }
            carry[grp] = 0.f;
            continue;
          }
          float vs[4] = {0.f, 0.f, 0.f, 0.f};
          float pr[16];
#pragma unroll
          for (int r = 0; r < 16; ++r) {
            float p = fast_exp2(fmaf(__uint_as_float(v16[r]), sl2, -lse16[r]));
            if (MASKED && (j > ig + r || j < 0)) p = 0.f;
            vs[r & 3] += p;
            pr[r] = p;
          }
          // the scores of the next group travel from TMEM while this group's diagonals are summed
          if (grp + 1 < RS_PROBE_GROUPS) tmem_ld16(t_hh + (uint32_t)(grp + 1) * 16u, v16);
          if (store && j < q1) vert_h[(size_t)grp * P.n + j] = (vs[0] + vs[1]) + (vs[2] + vs[3]);
          // Diagonal sums by lane rotation: the diagonal that ends at this thread's key takes row r from the key
          // 15 - r to the left.  One rotation per row serves both ends: lanes >= 15 - r receive an entry of their own
          // diagonal, the lanes below receive (wrapped around) the entry that belongs to the diagonal ending at the
          // same lane of the NEXT 32 keys, i.e. the carry into the warp's next step.
          float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int r = 0; r < 16; ++r) {
            const int sh = 15 - r;
            const float t = sh == 0 ? pr[r] : __shfl_sync(0xffffffffu, pr[r], (lane - sh) & 31);
            if (lane >= sh) acc0[r & 3] += t;
            else acc1[r & 3] += t;
          }
          const int o = ig + 15 - j;                    // the offset whose diagonal ends at this key
          if (store) {
            if (o >= 0) slash_h[(size_t)grp * P.n + o] = ((acc0[0] + acc0[1]) + (acc0[2] + acc0[3])) + carry[grp];
            else if (j < q1) slash_h[(size_t)grp * P.n + j] = 0.f;
          }
          carry[grp] = (acc1[0] + acc1[1]) + (acc1[2] + acc1[3]);     // zero in lanes 15 and above
        }
      };
      for (int it = 0; it < n_mma; ++it) {
        const int b = it & 1;
        ok = mbar_wait(bar_tfull[b], (uint32_t)(it >> 1) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const int jw = key_q + (it - 1) * 32;           // first key of the step
        if (jw + 31 > i_min || jw < 0) step(std::true_type{}, b, jw, it > 0 && live);
        else step(std::false_type{}, b, jw, it > 0 && live);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty[b]);   // one arrival per warp: 512 arrivals per tile queue up on the barrier
      }
    }
    if (!ok && lane == 0) { rs_report(P.status, RS_ERR_TIMEOUT, 15); *abort_flag = 1; }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, kTmemCols); }
}

// 64-row means of Q (fp32), every block.
// One CTA per (tensor row block): 256 threads, thread (rg = tid/16, cc = tid%16) sums rows rg, rg+16, .. of 16-byte
// column chunk cc; a fixed-order shared-memory reduction over the 16 row groups follows.
__global__ void __launch_bounds__(256)
rs_pool_kernel(const __nv_bfloat16* __restrict__ X, float* __restrict__ out, long long n_blocks) {
  __shared__ float red[16][128 + 4];
  const long long blk = blockIdx.x;
  if (blk >= n_blocks) return;
  const int rg = threadIdx.x >> 4, cc = threadIdx.x & 15;
  const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)blk * 64 * RS_HEAD_DIM);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint4 u = __ldg(src + (size_t)(rg + 16 * k) * 16 + cc);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[2 * e] += __uint_as_float(w[e] << 16);
      acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[rg][cc * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < 128) {
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) sum += red[r][threadIdx.x];
    out[(size_t)blk * RS_HEAD_DIM + threadIdx.x] = sum * (1.0f / 64.0f);
  }
}

// Block maxima of ||v||^2: one CTA per 64-row block, 16 lanes per row.
__global__ void __launch_bounds__(256)
rs_vnorm_block_kernel(const __nv_bfloat16* __restrict__ V, float* __restrict__ blockmax, long long n_blocks) {
  __shared__ float red[8];
  const long long blk = blockIdx.x;
  if (blk >= n_blocks) return;
  const int rg = threadIdx.x >> 4, cc = threadIdx.x & 15;
  const uint4* src = reinterpret_cast<const uint4*>(V + (size_t)blk * 64 * RS_HEAD_DIM);
  float best = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint4 u = __ldg(src + (size_t)(rg + 16 * k) * 16 + cc);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = __uint_as_float(w[e] << 16), b = __uint_as_float(w[e] & 0xffff0000u);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
    // 16 lanes hold one row: fixed-order butterfly
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    best = fmaxf(best, ss);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
    blockmax[blk] = m;
  }
}

struct ProbePlan { size_t partial, blockmax, total; int n_units, n_splits, n_hc, per; };

ProbePlan plan(const rs_problem* p) {
  ProbePlan w{};
  const int group = p->n_q_heads / p->n_kv_heads;
  w.n_hc = (group + kHC - 1) / kHC;
  w.n_units = p->n_segments * p->n_kv_heads * w.n_hc;
  // Every CTA gets about the same number of key tiles: segments that end early have fewer tiles and use fewer CTAs
  // (two CTAs' worth of work per SM in total).
  const int per_seg_units = p->n_kv_heads * w.n_hc;
  long long total_tiles = 0;
  for (int s = 0; s < p->n_segments; ++s) total_tiles += (long long)per_seg_units * ((p->seg_bounds[s + 1] + kKeyTile - 1) / kKeyTile);
  const int max_tiles = (p->n_keys + kKeyTile - 1) / kKeyTile;
  int per = (int)((total_tiles + 2 * 148 - 1) / (2 * 148));
  if (per < 1) per = 1;
  if ((max_tiles + per - 1) / per > 64) per = (max_tiles + 63) / 64;
  const int splits = (max_tiles + per - 1) / per;
  w.per = per;
  w.n_splits = splits;
  size_t off = 0;
  w.partial = off;  off += rs_align_up((size_t)w.n_units * 2 * splits * kRows * sizeof(float4), 256);
  w.blockmax = off; off += rs_align_up((size_t)p->n_kv_heads * (p->n_keys / 64) * sizeof(float), 256);
  w.total = off;
  return w;
}

}  // namespace

size_t rs_probe_workspace_bytes(const rs_problem* p) { return plan(p).total; }

namespace {

// 64-row mean of one block (all 256 threads of the CTA); same arithmetic and summation order as rs_pool_kernel.
__device__ __forceinline__ void pool_block(const __nv_bfloat16* __restrict__ X, float* __restrict__ out, long long blk,
                                           float (*red)[128 + 4]) {
  const int rg = threadIdx.x >> 4, cc = threadIdx.x & 15;
  const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)blk * 64 * RS_HEAD_DIM);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint4 u = __ldg(src + (size_t)(rg + 16 * k) * 16 + cc);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[2 * e] += __uint_as_float(w[e] << 16);
      acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[rg][cc * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < 128) {
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) sum += red[r][threadIdx.x];
    out[(size_t)blk * RS_HEAD_DIM + threadIdx.x] = sum * (1.0f / 64.0f);
  }
}

// 64-row means of the Q blocks of the heads routed to block-sparse (every head without a choice), a run of kPoolRun
// consecutive query blocks per CTA: most heads are not routed to block-sparse, and tens of thousands of CTAs that
// leave at once still cost a tenth of a millisecond to launch.  Same arithmetic and summation order as rs_pool_kernel.
constexpr int kPoolRun = 32;
__global__ void __launch_bounds__(256)
rs_pool_q_routed_kernel(ProbeParams P, const __nv_bfloat16* __restrict__ Q, float* __restrict__ out, rs_candidate_list L,
                        const int32_t* __restrict__ choice) {
  __shared__ float red[16][128 + 4];
  const int nb = P.n >> 6;
  const int h = blockIdx.y;
  int s = -1;
  bool want = false;
  for (int qb = blockIdx.x * kPoolRun; qb < min(nb, (int)(blockIdx.x + 1) * kPoolRun); ++qb) {
    if (s < 0 || qb * 64 >= P.seg_bounds[s + 1]) {          // the route is looked up once per segment of the run
      s = max(s, 0);
      while (s + 1 < P.n_seg && qb * 64 >= P.seg_bounds[s + 1]) ++s;
      want = choice == nullptr || L.pattern[choice[s * P.Hq + h]] == RS_BLOCK_SPARSE;
    }
    if (!want) continue;                                    // uniform over the CTA
    pool_block(Q, out, (long long)h * nb + qb, red);
    __syncthreads();
  }
}


}  // namespace

extern "C" int rs_pool_queries(const rs_problem* p, const void* Q, const rs_candidate* lib, int n_cand,
                               const int32_t* choice, float* qpool, int32_t* status, void* stream_) {
  (void)status;
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !qpool || n_cand < 0 || n_cand > RS_MAX_CANDIDATES || (choice != nullptr && (!lib || n_cand == 0)))
    return RS_ERR_INVALID_ARG;
  rc = rs_check_device();
  if (rc != RS_OK) return rc;
  ProbeParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = P.Hq / P.Hkv; P.n_seg = p->n_segments;
  for (int s = 0; s <= p->n_segments; ++s) P.seg_bounds[s] = p->seg_bounds[s];
  rs_candidate_list L{};
  bool any_bs = choice == nullptr;
  for (int c = 0; c < n_cand; ++c) { L.pattern[c] = lib[c].pattern; any_bs |= lib[c].pattern == RS_BLOCK_SPARSE; }
  if (!any_bs) return RS_OK;                            // no block-sparse candidate: nothing can be routed to it
  const int nb = P.n >> 6;
  rs_pool_q_routed_kernel<<<dim3((nb + kPoolRun - 1) / kPoolRun, P.Hq), 256, 0, (cudaStream_t)stream_>>>(
      P, reinterpret_cast<const __nv_bfloat16*>(Q), qpool, L, choice);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

// rs_probe and rs_probe_runs.  run_starts: host int32 [n_seg][4], first row of each 16-row group of probe rows, or
// NULL for the last 64 rows of every segment.
static int probe_impl(const rs_problem* p, const void* Q, const void* K, const void* V, const int32_t* run_starts,
                      float* vert, float* slash, float* lse_probe, float* qpool, float* kpool, float* vmax, float* descr,
                      int flags, void* ws, size_t ws_bytes, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !K || !V || !vert || !slash || !lse_probe || !ws) return RS_ERR_INVALID_ARG;
  for (int s = 0; s < p->n_segments; ++s) {
    if (p->seg_bounds[s + 1] < RS_PROBE_ROWS) return RS_ERR_UNSUPPORTED_SHAPE;
    for (int g = 0; run_starts != nullptr && g < RS_PROBE_GROUPS; ++g) {
      const int r0 = run_starts[s * RS_PROBE_GROUPS + g];
      if (r0 < 0 || r0 + 16 > p->seg_bounds[s + 1]) return RS_ERR_INVALID_ARG;
    }
  }
  rc = rs_check_device();
  if (rc != RS_OK) return rc;
  const ProbePlan w = plan(p);
  if (ws_bytes < w.total) return RS_ERR_WORKSPACE_TOO_SMALL;
  if (((uintptr_t)ws & 255) != 0) return RS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);

  ProbeParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = P.Hq / P.Hkv;
  P.n_seg = p->n_segments; P.n_hc = w.n_hc; P.n_splits = w.n_splits; P.per = w.per;
  for (int s = 0; s <= p->n_segments; ++s) P.seg_bounds[s] = p->seg_bounds[s];
  for (int s = 0; s < p->n_segments; ++s)
    for (int g = 0; g < RS_PROBE_GROUPS; ++g)
      P.run_start[s][g] = run_starts ? run_starts[s * RS_PROBE_GROUPS + g] : p->seg_bounds[s + 1] - RS_PROBE_ROWS + 16 * g;
  P.partial = reinterpret_cast<float4*>(wsb + w.partial);
  P.descr = descr;
  P.lse_probe = lse_probe; P.vert = vert; P.slash = slash; P.kpool = kpool; P.status = status;
  P.scale_log2e = (float)(1.4426950408889634 / sqrt((double)RS_HEAD_DIM));

  // Pass 2 writes every entry below a segment's end exactly once; what lies beyond the end of a segment that stops
  // before n_keys is zero by definition and is cleared here (nothing to do for a single segment).
  for (int s = 0; s < P.n_seg; ++s) {
    const int q1 = P.seg_bounds[s + 1];
    if (q1 >= P.n) continue;
    const size_t rows = (size_t)P.Hq * RS_PROBE_GROUPS, first = (size_t)s * rows * (size_t)P.n + (size_t)q1;
    const size_t pitch = (size_t)P.n * sizeof(float), width = (size_t)(P.n - q1) * sizeof(float);
    if (cudaMemset2DAsync(vert + first, pitch, 0, width, rows, stream) != cudaSuccess ||
        cudaMemset2DAsync(slash + first, pitch, 0, width, rows, stream) != cudaSuccess)
      return RS_ERR_CUDA;
  }

  CUtensorMap tmQ, tmK, tmK32;      // K in boxes of 128 keys (pass 1) and of 32 keys (pass 2: one box per lane quadrant)
  if (rs_make_tmap_bf16_2d(&tmQ, Q, (uint64_t)P.Hq * P.n, RS_HEAD_DIM, 16, 64) ||      // one box per group of probe rows
      rs_make_tmap_bf16_2d(&tmK, K, (uint64_t)P.Hkv * P.n, RS_HEAD_DIM, kKeyTile, 64) ||
      rs_make_tmap_bf16_2d(&tmK32, K, (uint64_t)P.Hkv * P.n, RS_HEAD_DIM, 32, 64))
    return RS_ERR_CUDA;
  static rs_smem_attr attr_pass1, attr_pass2;
  if (rs_ensure_dynamic_smem(attr_pass1, rs_probe_kernel<1>, (int)SmemT<1>::total) != RS_OK ||
      rs_ensure_dynamic_smem(attr_pass2, rs_probe_kernel<2>, (int)SmemT<2>::total) != RS_OK)
    return RS_ERR_CUDA;
  // Pass 1 also pools K; pass 2 turns the block maxima of ||v||^2 into vmax and pools the last query block of every
  // segment from the probe rows it stages.  The block maxima only read V, the pooling of every query block (when it
  // is asked for) only Q: they run beside the passes on the side stream.  Pass 1 is enqueued first so that its CTAs
  // (one per SM, most of the shared memory) are resident before the small streaming CTAs fill what is left; the
  // other way round the streaming kernels would run alone.
  const long long nb = p->n_keys / 64;
  const bool pool_all = qpool != nullptr && !(flags & RS_PROBE_QPOOL_LAST_ONLY);
  if (qpool && !pool_all) P.qpool_last = qpool;
  const bool use_side = vmax != nullptr || pool_all;
  cudaStream_t side = nullptr;
  if (use_side) {
    rc = rs_side_fork(stream, &side);
    if (rc != RS_OK) return rc;
  }
  dim3 grid(w.n_splits, w.n_units);
  rs_probe_kernel<1><<<grid, kThreads1, SmemT<1>::total, stream>>>(tmQ, tmK, P);
  if (vmax) {
    float* blockmax = reinterpret_cast<float*>(wsb + w.blockmax);
    rs_vnorm_block_kernel<<<(unsigned)(P.Hkv * nb), 256, 0, side>>>(reinterpret_cast<const __nv_bfloat16*>(V), blockmax, P.Hkv * nb);
    P.blockmax = blockmax; P.vmax = vmax;
    rc = rs_side_sync_here(stream);          // pass 2 reads the block maxima (they are long done when pass 1 ends)
    if (rc != RS_OK) { rs_side_join(stream); return rc; }
  }
  if (pool_all)
    rs_pool_kernel<<<(unsigned)(P.Hq * nb), 256, 0, side>>>(reinterpret_cast<const __nv_bfloat16*>(Q), qpool, P.Hq * nb);
  rs_probe_kernel<2><<<grid, kThreads2, SmemT<2>::total, stream>>>(tmQ, tmK32, P);
  if (use_side) {
    rc = rs_side_join(stream);
    if (rc != RS_OK) return rc;
  }
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

extern "C" int rs_probe(const rs_problem* p, const void* Q, const void* K, const void* V, float* vert, float* slash,
                        float* lse_probe, float* qpool, float* kpool, float* vmax, float* descr, int flags, void* ws,
                        size_t ws_bytes, int32_t* status, void* stream) {
  return probe_impl(p, Q, K, V, nullptr, vert, slash, lse_probe, qpool, kpool, vmax, descr, flags, ws, ws_bytes, status, stream);
}

extern "C" int rs_probe_runs(const rs_problem* p, const void* Q, const void* K, const int32_t* run_starts, float* vert,
                             float* slash, float* lse_probe, void* ws, size_t ws_bytes, int32_t* status, void* stream) {
  if (run_starts == nullptr) return RS_ERR_INVALID_ARG;
  // V is only read by the value-norm kernel, which does not run here; K stands in for the argument check
  return probe_impl(p, Q, K, K, run_starts, vert, slash, lse_probe, nullptr, nullptr, nullptr, nullptr, 0, ws, ws_bytes,
                    status, stream);
}
