// Candidate index construction, coverage and pair counts (Section 3.1, 3.2; step 2 of the per-layer procedure).
//
// Everything that decides an index is integer arithmetic so that the result does not depend on the order of
// evaluation: ranking keys are sum_g floor(mass_g * 2^32) (uint64), top-k is "key descending, index ascending"
// found by an exact radix select (threshold key + quota of ties in index order) followed by an ordered
// compaction, coverage is a sum of the same fixed-point values, and pair counts are closed forms.
// Block-sparse scores are fp32 (fused pooled dot products accumulated k = 0..127 with fmaf, or an explicit
// score matrix) compared through an order-preserving integer transform.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

typedef unsigned long long u64;

struct IdxParams {
  int n, Hq, Hkv, group, n_seg, n_cand, nb;
  int seg_bounds[RS_MAX_SEGMENTS + 1];
  rs_candidate lib[RS_MAX_CANDIDATES];
  const float* vert; const float* slash; const float* qpool; const float* kpool; const float* bscore;
  const float* rank_vert; const float* rank_slash;   // masses the line lists are ranked by (== vert / slash unless given)
  const int32_t* choice;
  rs_index_set out;
  rs_cand_stats* stats;
  u64* vblk;          // [n_items][4][nb] block sums of fx(vert)
  float* bs_ws;       // [Hq][nb][nb] fused block scores (materialise mode)
  u64* keys;          // [n_items][2][n] ranking keys of columns (0) and offsets (1)
  float* bs_eval_ws;  // [n_items][nb] pooled scores of each segment's last query block
  int32_t* status;
  float scale;
};

// floor(x * 2^32) of a non-negative float, exactly: the scaling by a power of two is exact in fp32 (the masses are far
// below 2^95) and the conversion rounds toward zero.
__device__ __forceinline__ u64 fx(float x) {
  return __float2ull_rz(x * 4294967296.0f);
}

// Adds v of every thread of the block to *target (shared memory): the warp sums first, so that one 64-bit atomic per
// warp reaches the word (hundreds of threads on one shared 64-bit word serialise in a compare-and-swap loop).
// Integer addition: the result does not depend on the order.  All threads of the warp must call it.
__device__ __forceinline__ void warp_sum_then_add(u64 v, u64* target) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  if ((threadIdx.x & 31) == 0 && v != 0) atomicAdd(target, v);
}

__device__ __forceinline__ u64 line_key(const float* mass, int n, int j) {
  return fx(mass[j]) + fx(mass[(size_t)n + j]) + fx(mass[2 * (size_t)n + j]) + fx(mass[3 * (size_t)n + j]);
}

__device__ __forceinline__ int seg_of_block(const IdxParams& P, int qb) {
  int s = 0;
  while (s + 1 < P.n_seg && qb * 64 >= P.seg_bounds[s + 1]) ++s;
  return s;
}

// job -> (item, candidate, slot); returns false when this block has nothing to do
__device__ __forceinline__ bool job_of(const IdxParams& P, int job, int& item, int& c, int& slot) {
  item = job / P.n_cand;
  c = job - item * P.n_cand;
  if (P.choice != nullptr) {
    if (P.choice[item] != c) return false;
    slot = item;
  } else {
    slot = job;
  }
  return true;
}

// ------------------------------------------------------------------------------------------ block sums of fx(vert)
__global__ void rs_vblk_kernel(IdxParams P) {
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int total = P.n_seg * P.Hq * RS_PROBE_GROUPS * P.nb;
  if (warp_global >= total) return;
  const int kb = warp_global % P.nb;
  const int ig = warp_global / P.nb;            // item * 4 + g
  const int item = ig >> 2;
  const int s = item / P.Hq;
  u64 acc = 0;
  if (kb * 64 < P.seg_bounds[s + 1]) {
    const float* src = P.vert + (size_t)ig * P.n + (size_t)kb * 64;
    acc = fx(src[lane]) + fx(src[lane + 32]);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) P.vblk[(size_t)ig * P.nb + kb] = acc;
}

// ------------------------------------------------------------------------------------------ ranking keys, once per line
// With fuse_vblk the blocks of list 0 also write the 64-key block sums of fx(vert) (what rs_vblk_kernel computes):
// they hold the four fixed-point values of every key anyway.
__global__ void __launch_bounds__(256)
rs_vs_keys_kernel(IdxParams P, int fuse_vblk) {
  __shared__ u64 half_sum[8][RS_PROBE_GROUPS];
  const int item = blockIdx.y >> 1, list = blockIdx.y & 1;
  const int s = item / P.Hq;
  const int q1 = P.seg_bounds[s + 1];
  const int j = blockIdx.x * 256 + threadIdx.x;
  const float* mass = (list == 0 ? P.rank_vert : P.rank_slash) + (size_t)item * RS_PROBE_GROUPS * P.n;
  u64 f[RS_PROBE_GROUPS] = {0, 0, 0, 0};
  if (j < q1) {
#pragma unroll
    for (int g = 0; g < RS_PROBE_GROUPS; ++g) f[g] = fx(mass[(size_t)g * P.n + j]);
    P.keys[((size_t)item * 2 + list) * P.n + j] = (f[0] + f[1]) + (f[2] + f[3]);
  }
  if (!fuse_vblk || list != 0) return;                  // uniform over the block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int g = 0; g < RS_PROBE_GROUPS; ++g) {
    u64 v = f[g];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    if (lane == 0) half_sum[warp][g] = v;
  }
  __syncthreads();
  if (threadIdx.x < 4 * RS_PROBE_GROUPS) {
    const int blk = threadIdx.x >> 2, g = threadIdx.x & 3;
    const int kb = blockIdx.x * 4 + blk;
    if (kb < P.nb) P.vblk[((size_t)item * RS_PROBE_GROUPS + g) * P.nb + kb] = half_sum[2 * blk][g] + half_sum[2 * blk + 1][g];
  }
}

// ------------------------------------------------------------------------------------------ exact top-k of a line list
// grid = (kSelCluster, 2 lists x items, groups of up to kSelMaxC vertical-slash candidates); the kSelCluster blocks of
// a thread-block cluster share one list: block r owns the r-th contiguous eighth of the domain.  list 0: vertical
// columns over [0, q1); list 1: slash offsets over [1, q1) plus offset 0.  A cluster serves every budget of its group
// in the same passes over the keys: per radix digit every block histograms its own eighth into shared memory, the
// blocks read each other's histograms through distributed shared memory (integer counts: the sum does not depend on the
// order) and each one locates the k-th entry itself; one counting sweep plus one writing sweep produce the ordered
// lists, the position of a block's first entry being the number of entries the lower-ranked blocks select.
constexpr int kSelCluster = 8;
constexpr int kSelThreads = 256;  // small blocks: all clusters of a layer (2 lists x 32 items x 8 blocks) are resident at once
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kDigitBits = 11;    // four digits cover 44 bits; ranking keys stay below 2^39
constexpr int kSelPasses = 4;
constexpr int kBins = 1 << kDigitBits;
constexpr int kSlice = kBins / kSelCluster;      // bins of a histogram that one block of the cluster scans
static_assert(kSlice == kSelThreads, "one bin per thread");
constexpr int kSelMaxC = 4;       // budgets served by one cluster: four histograms are 32 KB of shared memory per block
constexpr int kSelBatch = 8;      // independent key loads in flight per thread

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads, 4)
rs_vs_select_kernel(IdxParams P) {
  extern __shared__ unsigned int sel_hist[];             // [unique prefixes <= kSelMaxC][kBins]
  __shared__ unsigned int wsum[kSelMaxC * kSelWarps];
  __shared__ u64 sh_prefix[kSelMaxC], nx_prefix[kSelMaxC];
  __shared__ unsigned int sh_k[kSelMaxC], nx_k[kSelMaxC];
  __shared__ unsigned int slice_tot[kSelMaxC];           // entries in this block's slice of the bins
  __shared__ unsigned int w_gt[kSelMaxC][kSelWarps], w_eq[kSelMaxC][kSelWarps];
  __shared__ unsigned int cta_tot[2 * kSelMaxC];         // this block's entries above / equal to each threshold
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int list = blockIdx.y & 1, item = blockIdx.y >> 1;
  // the vertical-slash candidates this cluster serves
  int cand_id[kSelMaxC] = {}, slot_id[kSelMaxC] = {}, kk[kSelMaxC] = {};
  int nC = 0;
  {
    int seen = 0;
    for (int c = 0; c < P.n_cand; ++c) {
      if (P.lib[c].pattern != RS_VERTICAL_SLASH) continue;
      if (P.choice != nullptr && P.choice[item] != c) continue;
      if (seen / kSelMaxC == (int)blockIdx.z && nC < kSelMaxC) {
        const int sl = (P.choice != nullptr) ? item : item * P.n_cand + c;
        _Pragma("unroll") for (int e = 0; e < kSelMaxC; ++e) if (e == nC) { cand_id[e] = c; slot_id[e] = sl; }
        ++nC;
      }
      ++seen;
    }
  }
  if (nC == 0) return;                                   // the same for every block of the cluster
  const int s = item / P.Hq;
  const int q1 = P.seg_bounds[s + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u64* keys = P.keys + ((size_t)item * 2 + list) * P.n;
  const int first = (list == 0) ? 0 : 1;                 // first index of the domain
  const int n_dom = q1 - first;
  _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
    const rs_candidate cand = P.lib[cand_id[c]];
    int k = (list == 0) ? min(cand.b0, q1) : (min(cand.b1, q1) - 1);
    if (k < 0) k = 0;
    if (k > n_dom) k = n_dom;
    kk[c] = k;
  }
  const int cap = (list == 0) ? P.out.kv_cap : P.out.ks_cap;
  // this block's part of the domain: [c_lo, c_hi)
  const int c_len = (((n_dom + kSelCluster - 1) / kSelCluster) + 31) / 32 * 32;
  const int c_lo = min(n_dom, rank * c_len), c_hi = min(n_dom, c_lo + c_len);
  const unsigned int* rhist[kSelCluster];
#pragma unroll
  for (int r = 0; r < kSelCluster; ++r) rhist[r] = cluster.map_shared_rank(sel_hist, r);

  // ---- thresholds: T[c] = key of the k-th entry in "key descending" order, k_eq[c] = how many of its ties are taken
  if (tid < nC) { sh_prefix[tid] = 0; sh_k[tid] = (unsigned)kk[tid]; }
  __syncthreads();
  for (int pass = kSelPasses - 1; pass >= 0; --pass) {
    const int shift = pass * kDigitBits;
    // candidates with the same prefix share a histogram: hsel[c] = index of the first candidate with that prefix
    u64 pre[kSelMaxC];
    int hsel[kSelMaxC];
    int n_hist = 0;
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
      pre[c] = sh_prefix[c];
      hsel[c] = -1;
      if (kk[c] == 0) continue;
      _Pragma("unroll") for (int d = 0; d < kSelMaxC; ++d)
        if (d < c && hsel[c] < 0 && kk[d] > 0 && pre[d] == pre[c]) hsel[c] = hsel[d];
      if (hsel[c] < 0) hsel[c] = n_hist++;
    }
    for (int i = tid; i < n_hist * kBins; i += kSelThreads) sel_hist[i] = 0;
    // the distinct prefixes, in histogram order: a key matches at most one of them (what lies above this digit fits
    // 32 bits: keys stay below 2^39 and every prefix has lost at least 11 bits)
    uint32_t upre[kSelMaxC];
    _Pragma("unroll") for (int u = 0; u < kSelMaxC; ++u) {
      upre[u] = 0xffffffffu;
      _Pragma("unroll") for (int c = kSelMaxC - 1; c >= 0; --c) if (c < nC && hsel[c] == u) upre[u] = (uint32_t)pre[c];
    }
    __syncthreads();
    // eight independent loads per thread are in flight before any is used: the sweep is latency-bound otherwise
    for (int base = c_lo; base < c_hi; base += kSelThreads * kSelBatch) {
      u64 keyb[kSelBatch];
      bool inb[kSelBatch];
#pragma unroll
      for (int u = 0; u < kSelBatch; ++u) {
        const int j = base + u * kSelThreads + tid;
        inb[u] = j < c_hi;
        keyb[u] = inb[u] ? keys[first + j] : 0ull;
      }
#pragma unroll
      for (int u = 0; u < kSelBatch; ++u) {
        const uint32_t hi = (uint32_t)(keyb[u] >> (shift + kDigitBits));
        const uint32_t dig = (uint32_t)(keyb[u] >> shift) & (kBins - 1);
        unsigned int slot = 0xffffffffu;                 // histogram * kBins + digit, or none
        _Pragma("unroll") for (int h = 0; h < kSelMaxC; ++h)
          if (hi == upre[h]) slot = (unsigned)h * kBins + dig;
        if (!inb[u]) slot = 0xffffffffu;
        if (__ballot_sync(0xffffffffu, slot != 0xffffffffu) == 0u) continue;   // nobody in this warp matches a prefix
        // the upper digits of most keys are equal (small masses): one addition for the warp when all 32 agree,
        // one per lane otherwise (in the lower digits the lanes rarely meet)
        const unsigned int slot0 = __shfl_sync(0xffffffffu, slot, 0);
        if (__all_sync(0xffffffffu, slot == slot0)) {
          if (lane == 0) atomicAdd(&sel_hist[slot], 32u);
        } else if (slot != 0xffffffffu) {
          atomicAdd(&sel_hist[slot], 1u);
        }
      }
    }
    cluster.sync();                                      // every block's histogram of this digit is complete
    // Block r owns the bins [1024 r, 1024 r + 1024) of every histogram: thread t sums bin 1024 r + 1023 - t over the
    // blocks of the cluster (counts: the order does not matter) and the block scans its slice from the top.
    unsigned int v[kSelMaxC], incl[kSelMaxC];
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) {
      v[c] = 0; incl[c] = 0;
      if (c >= nC || kk[c] == 0) continue;               // uniform over the cluster
      const int bin = kSlice * rank + (kSlice - 1 - tid);
      unsigned int sum = 0;
#pragma unroll
      for (int r = 0; r < kSelCluster; ++r) sum += rhist[r][hsel[c] * kBins + bin];
      v[c] = sum;
      unsigned int in = sum;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, in, off);
        if (lane >= off) in += t;
      }
      if (lane == 31) wsum[c * kSelWarps + warp] = in;
      incl[c] = in;
    }
    __syncthreads();
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) {
      if (c >= nC || kk[c] == 0) continue;
      unsigned int before = 0;
      for (int w = 0; w < warp; ++w) before += wsum[c * kSelWarps + w];
      incl[c] += before;
      if (tid == kSelThreads - 1) slice_tot[c] = incl[c];
    }
    cluster.sync();                                      // every block's slice totals are published
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) {
      if (c >= nC || kk[c] == 0) continue;
      unsigned int above = incl[c] - v[c];               // entries in higher bins: of this slice, and of the higher slices
      for (int r = rank + 1; r < kSelCluster; ++r) above += cluster.map_shared_rank(slice_tot, r)[c];
      const unsigned int kq = sh_k[c];
      if (above < kq && kq <= above + v[c]) {            // exactly one thread of the cluster: its bin holds the k-th entry
        const u64 new_prefix = (pre[c] << kDigitBits) | (u64)(kSlice * rank + (kSlice - 1 - tid));
        for (int r = 0; r < kSelCluster; ++r) {
          cluster.map_shared_rank(nx_prefix, r)[c] = new_prefix;
          cluster.map_shared_rank(nx_k, r)[c] = kq - above;
        }
      }
    }
    cluster.sync();                                      // the result has reached every block; this digit's histograms are done
    if (tid < nC && kk[tid] > 0) { sh_prefix[tid] = nx_prefix[tid]; sh_k[tid] = nx_k[tid]; }
    __syncthreads();
  }
  u64 T[kSelMaxC];
  unsigned int k_eq[kSelMaxC];
  _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
    T[c] = (kk[c] > 0) ? sh_prefix[c] : ~0ull;           // k = 0: nothing is above or equal
    k_eq[c] = (kk[c] > 0) ? sh_k[c] : 0u;
  }

  // ---- ordered compaction: warp w of block r walks the contiguous range [c_lo + w * chunk, c_lo + (w + 1) * chunk)
  const int chunk = (((c_hi - c_lo + kSelWarps - 1) / kSelWarps) + 31) / 32 * 32;
  const int lo = min(c_hi, c_lo + warp * chunk), hi = min(c_hi, lo + chunk);
  unsigned int gt[kSelMaxC], eq[kSelMaxC];
  _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) { gt[c] = 0; eq[c] = 0; }
  for (int base = lo; base < hi; base += 32 * kSelBatch) {
    u64 keyb[kSelBatch];
    bool inb[kSelBatch];
#pragma unroll
    for (int u = 0; u < kSelBatch; ++u) {
      const int j = base + u * 32 + lane;
      inb[u] = j < hi;
      keyb[u] = inb[u] ? keys[first + j] : 0ull;
    }
#pragma unroll
    for (int u = 0; u < kSelBatch; ++u) {
      if (inb[u]) {                                      // per-lane counts; the warp sums them once, after the sweep
        _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
          gt[c] += (keyb[u] > T[c]) ? 1u : 0u;
          eq[c] += (keyb[u] == T[c]) ? 1u : 0u;
        }
      }
    }
  }
  _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
    gt[c] = __reduce_add_sync(0xffffffffu, gt[c]);
    eq[c] = __reduce_add_sync(0xffffffffu, eq[c]);
  }
  if (lane == 0)
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) { w_gt[c][warp] = gt[c]; w_eq[c][warp] = eq[c]; }
  __syncthreads();
  if (tid < 2 * kSelMaxC) {
    const int c = tid >> 1;
    unsigned int tot = 0;
    if (c < nC) for (int w = 0; w < kSelWarps; ++w) tot += (tid & 1) ? w_eq[c][w] : w_gt[c][w];
    cta_tot[tid] = tot;
  }
  cluster.sync();                                        // every block's totals are published
  unsigned int pos[kSelMaxC], eq_run[kSelMaxC];
  _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
    unsigned int gt_before = 0, eq_before = 0;
    for (int r = 0; r < rank; ++r) {
      const unsigned int* rt = cluster.map_shared_rank(cta_tot, r);
      gt_before += rt[2 * c]; eq_before += rt[2 * c + 1];
    }
    for (int w = 0; w < warp; ++w) { gt_before += w_gt[c][w]; eq_before += w_eq[c][w]; }
    pos[c] = gt_before + min(k_eq[c], eq_before) + (list == 1 ? 1u : 0u);
    eq_run[c] = eq_before;
  }
  const unsigned int lt_mask = (1u << lane) - 1u;
  for (int base = lo; base < hi; base += 32 * kSelBatch) {
    u64 keyb[kSelBatch];
    bool inb[kSelBatch];
#pragma unroll
    for (int u = 0; u < kSelBatch; ++u) {
      const int j = base + u * 32 + lane;
      inb[u] = j < hi;
      keyb[u] = inb[u] ? keys[first + j] : 0ull;
    }
#pragma unroll
    for (int u = 0; u < kSelBatch; ++u) {
      const int j = base + u * 32 + lane;
      _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
        bool take = inb[u] && keyb[u] > T[c];
        if (__any_sync(0xffffffffu, inb[u] && keyb[u] == T[c])) {   // ties with the threshold are rare: taken in index order
          const bool is_eq = inb[u] && keyb[u] == T[c];
          const unsigned int beq = __ballot_sync(0xffffffffu, is_eq);
          take = take || (is_eq && eq_run[c] + __popc(beq & lt_mask) < k_eq[c]);
          eq_run[c] += __popc(beq);
        }
        const unsigned int bt = __ballot_sync(0xffffffffu, take);
        if (take) {
          const unsigned int p = pos[c] + __popc(bt & lt_mask);
          int32_t* out = (list == 0) ? (P.out.vs_cols + (size_t)slot_id[c] * P.out.kv_cap)
                                     : (P.out.vs_offs + (size_t)slot_id[c] * P.out.ks_cap);
          if ((int)p < cap) out[p] = first + j;
        }
        pos[c] += __popc(bt);
      }
    }
  }
  if (tid == 0 && rank == 0) {
    _Pragma("unroll") for (int c = 0; c < kSelMaxC; ++c) if (c < nC) {
      if (list == 1) {
        P.out.vs_offs[(size_t)slot_id[c] * P.out.ks_cap] = 0;
        P.out.vs_count[4 * slot_id[c] + 1] = kk[c] + 1;
      } else {
        P.out.vs_count[4 * slot_id[c] + 0] = kk[c];
      }
    }
  }
  cluster.sync();                                        // no block leaves while its totals may still be read
}

// ------------------------------------------------------------------------------------------ pair counts (closed forms)
__device__ __forceinline__ u64 pairs_dense(long long q0, long long q1) { return (u64)((q1 * (q1 + 1) - q0 * (q0 + 1)) / 2); }

__device__ __forceinline__ u64 pairs_a_shape(long long q0, long long q1, long long cap) {
  // sum_{i=q0}^{q1-1} min(i + 1, cap)
  const long long m = min(q1, max(q0, cap));            // rows [q0, m) have i + 1 <= cap
  u64 total = (u64)((m * (m + 1) - q0 * (q0 + 1)) / 2);
  total += (u64)((q1 - m) * cap);
  return total;
}

__device__ __forceinline__ u64 pairs_block_sparse(int qb_lo, int qb_hi, int k_b) {
  u64 total = 0;
  for (int qb = qb_lo; qb < qb_hi; ++qb) total += (u64)(min(k_b, qb + 1) - 1) * 4096ull + 2080ull;
  return total;
}

// ------------------------------------------------------------------------------------------ vertical-slash: D, coverage, pairs
constexpr int kFinishThreads = 512;
__device__ __forceinline__ void vs_finish_block(const IdxParams& P, int job) {
  __shared__ uint32_t dbits[128];
  __shared__ int wpre[129];
  __shared__ u64 cov[RS_PROBE_GROUPS];
  __shared__ u64 extra_pairs;
  int item, c, slot;
  if (!job_of(P, job, item, c, slot)) return;
  const rs_candidate cand = P.lib[c];
  if (cand.pattern != RS_VERTICAL_SLASH) return;
  const int s = item / P.Hq;
  const int q0 = P.seg_bounds[s], q1 = P.seg_bounds[s + 1];
  const int nbs = q1 >> 6, qb_lo = q0 >> 6, qb_star = nbs - 1;
  const int tid = threadIdx.x;
  const int n_cols = P.out.vs_count[4 * slot + 0], n_offs = P.out.vs_count[4 * slot + 1];
  const int32_t* cols = P.out.vs_cols + (size_t)slot * P.out.kv_cap;
  const int32_t* offs = P.out.vs_offs + (size_t)slot * P.out.ks_cap;
  int32_t* diag = P.out.vs_diag + (size_t)slot * P.out.nd_cap;
  for (int i = tid; i < 128; i += blockDim.x) dbits[i] = 0;
  if (tid < RS_PROBE_GROUPS) cov[tid] = 0;
  if (tid == 0) extra_pairs = 0;
  __syncthreads();
  for (int base = 0; base < n_offs; base += 8 * (int)blockDim.x) {     // eight independent loads in flight per thread
    int ob[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + u * (int)blockDim.x + tid;
      ob[u] = (i < n_offs) ? offs[i] : -1;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      // offsets are ascending, so the lanes of a warp see runs of equal block diagonals: only the first lane of a run
      // touches the bitmap (32 lanes hammering one shared-memory word would serialise)
      const int d0 = ob[u] < 0 ? -1 : ob[u] >> 6, d1 = ob[u] < 0 ? -1 : (ob[u] + 63) >> 6;
      const int p0 = __shfl_up_sync(0xffffffffu, d0, 1), p1 = __shfl_up_sync(0xffffffffu, d1, 1);
      const int lane = tid & 31;
      if (d0 >= 0 && d0 < nbs && (lane == 0 || p0 != d0)) atomicOr(&dbits[d0 >> 5], 1u << (d0 & 31));
      if (d1 >= 0 && d1 < nbs && d1 != d0 && (lane == 0 || p1 != d1)) atomicOr(&dbits[d1 >> 5], 1u << (d1 & 31));
    }
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int w = 0; w < 128; ++w) { wpre[w] = acc; acc += __popc(dbits[w]); }
    wpre[128] = acc;
  }
  __syncthreads();
  const int n_diag = wpre[128];
  if (tid < 128) {
    uint32_t bits = dbits[tid];
    int at = wpre[tid];
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if (at < P.out.nd_cap) diag[at] = tid * 32 + b;
      ++at;
    }
  }
  if (tid == 0) { P.out.vs_count[4 * slot + 2] = n_diag; P.out.vs_count[4 * slot + 3] = 0; }
  if (P.stats == nullptr) return;

  // coverage: block diagonals seen from the last query block + verticals outside them
  const float* vert = P.vert + (size_t)item * RS_PROBE_GROUPS * P.n;
  const u64* vblk = P.vblk + (size_t)item * RS_PROBE_GROUPS * P.nb;
  u64 part[RS_PROBE_GROUPS] = {0, 0, 0, 0};
  for (int kb = tid; kb < nbs; kb += blockDim.x) {
    const int d = qb_star - kb;
    if ((dbits[d >> 5] >> (d & 31)) & 1u) {
#pragma unroll
      for (int g = 0; g < RS_PROBE_GROUPS; ++g) part[g] += vblk[(size_t)g * P.nb + kb];
    }
  }
  // pairs: verticals not covered by a block diagonal of their query block
  u64 vp = 0;
  const bool has0 = (dbits[0] & 1u) != 0;
  // number of block diagonals of D with delta <= x, from the per-word prefix counts
  auto d_upto = [&](int x) -> int {
    if (x < 0) return 0;
    const int w = x >> 5;
    return wpre[w] + __popc(dbits[w] & (0xffffffffu >> (31 - (x & 31))));
  };
  for (int base = 0; base < n_cols; base += 4 * (int)blockDim.x) {      // four independent load chains per thread
    int jb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = base + u * (int)blockDim.x + tid;
      jb[u] = (i < n_cols) ? cols[i] : -1;
    }
    float vb[4][RS_PROBE_GROUPS];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = max(jb[u], 0);
#pragma unroll
      for (int g = 0; g < RS_PROBE_GROUPS; ++g) vb[u][g] = vert[(size_t)g * P.n + j];
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = jb[u];
      if (j < 0) continue;
      const int kbj = j >> 6;
      const int d = qb_star - kbj;
      if (!((dbits[d >> 5] >> (d & 31)) & 1u)) {
#pragma unroll
        for (int g = 0; g < RS_PROBE_GROUPS; ++g) part[g] += fx(vb[u][g]);
      }
      // query blocks qb in [max(kbj, qb_lo), nbs): delta = qb - kbj
      if (kbj >= qb_lo && !has0) vp += (u64)((kbj + 1) * 64 - j);
      const int d_lo = max(1, qb_lo - kbj), d_hi = qb_star - kbj;     // deltas >= 1 of the other query blocks
      if (d_hi >= d_lo) {
        const int covered = d_upto(d_hi) - d_upto(d_lo - 1);          // |D intersect [d_lo, d_hi]|
        vp += 64ull * (u64)(d_hi - d_lo + 1 - covered);
      }
    }
  }
#pragma unroll
  for (int g = 0; g < RS_PROBE_GROUPS; ++g) warp_sum_then_add(part[g], &cov[g]);
  if (tid < 128) {
    // block diagonals: delta >= 1 is used by every query block qb >= delta of the segment, delta 0 by all
    uint32_t bits = dbits[tid];
    while (bits) {
      const int d = tid * 32 + __ffs(bits) - 1;
      bits &= bits - 1;
      if (d == 0) vp += (u64)(nbs - qb_lo) * 2080ull;
      else if (nbs > max(qb_lo, d)) vp += (u64)(nbs - max(qb_lo, d)) * 4096ull;
    }
  }
  warp_sum_then_add(vp, &extra_pairs);
  __syncthreads();
  if (tid == 0) {
    rs_cand_stats* st = P.stats + (size_t)item * P.n_cand + c;
    for (int g = 0; g < RS_PROBE_GROUPS; ++g) st->cov_fx[g] = cov[g];
    st->pairs = extra_pairs;
  }
}

// ------------------------------------------------------------------------------------------ A-shape and dense stats
__device__ __forceinline__ void simple_stats_block(const IdxParams& P, int job) {
  __shared__ u64 cov[RS_PROBE_GROUPS];
  int item, c, slot;
  if (!job_of(P, job, item, c, slot)) return;
  if (P.stats == nullptr) return;
  const rs_candidate cand = P.lib[c];
  if (cand.pattern != RS_A_SHAPE && cand.pattern != RS_DENSE) return;
  const int s = item / P.Hq;
  const int q0 = P.seg_bounds[s], q1 = P.seg_bounds[s + 1];
  rs_cand_stats* st = P.stats + (size_t)item * P.n_cand + c;
  const int tid = threadIdx.x;
  if (cand.pattern == RS_DENSE) {
    if (tid == 0) {
      for (int g = 0; g < RS_PROBE_GROUPS; ++g) st->cov_fx[g] = 16ull << 32;
      st->pairs = pairs_dense(q0, q1);
    }
    return;
  }
  if (tid < RS_PROBE_GROUPS) cov[tid] = 0;
  __syncthreads();
  const float* vert = P.vert + (size_t)item * RS_PROBE_GROUPS * P.n;
  const float* slash = P.slash + (size_t)item * RS_PROBE_GROUPS * P.n;
  const int n_sink = cand.b0, win = cand.b1;
  const bool window_covers_all = win >= q1;
  const int n_off = window_covers_all ? q1 : win;
  const int n_col = window_covers_all ? 0 : min(n_sink, q1);
  u64 part[RS_PROBE_GROUPS] = {0, 0, 0, 0};
#pragma unroll 4
  for (int o = tid; o < n_off; o += blockDim.x)
#pragma unroll
    for (int g = 0; g < RS_PROBE_GROUPS; ++g) part[g] += fx(slash[(size_t)g * P.n + o]);
  for (int j = tid; j < n_col; j += blockDim.x)
#pragma unroll
    for (int g = 0; g < RS_PROBE_GROUPS; ++g) part[g] += fx(vert[(size_t)g * P.n + j]);
#pragma unroll
  for (int g = 0; g < RS_PROBE_GROUPS; ++g) warp_sum_then_add(part[g], &cov[g]);
  __syncthreads();
  if (tid == 0) {
    for (int g = 0; g < RS_PROBE_GROUPS; ++g) st->cov_fx[g] = cov[g];
    st->pairs = pairs_a_shape(q0, q1, (long long)n_sink + win);
  }
}

// ------------------------------------------------------------------------------------------ block-sparse row selection
__device__ __forceinline__ uint32_t f32_order_key(float x) {
  if (x == 0.f) x = 0.f;                     // -0 and +0 compare equal
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Selects the `take` largest of score[0, m) (ties -> lower index) plus the diagonal block `qb`; writes them
// ascending to out[] and returns the count.  All NT threads of the block call it; scores live in shared memory.
template <int NT>
__device__ int select_row(const float* score, int m, int take, int qb, int32_t* out, int cap, uint32_t* hist /*256*/,
                          uint32_t* sh /*8*/, unsigned int* wcnt /* 2 * NT / 32 */) {
  constexpr int NW = NT / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t T = 0xffffffffu, k_eq = 0;
  take = min(take, m);
  if (take > 0) {
    if (tid == 0) { sh[0] = 0; sh[1] = (uint32_t)take; }
    for (int pass = 3; pass >= 0; --pass) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      const uint32_t prefix = sh[0];
      const int shift = pass * 8;
      for (int i = tid; i < m; i += NT) {
        const uint32_t key = f32_order_key(score[i]);
        if (pass == 3 || (key >> (shift + 8)) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (warp == 0) {
        // the bin in which the count from the top reaches kk: eight bins per lane, counts above a lane by a suffix
        // scan over the lanes, then the one lane that holds the crossing walks its bins from the top
        const uint32_t kk = sh[1];
        uint32_t h8[8], local = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) { h8[b] = hist[8 * lane + b]; local += h8[b]; }
        uint32_t incl = local;                            // sum over lanes >= this one
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t o = __shfl_down_sync(0xffffffffu, incl, off);
          if (lane + off < 32) incl += o;
        }
        uint32_t acc = incl - local;
        __syncwarp();
        if (acc < kk && incl >= kk) {
#pragma unroll
          for (int b = 7; b >= 0; --b) {
            if (acc + h8[b] >= kk) { sh[0] = (prefix << 8) | (uint32_t)(8 * lane + b); sh[1] = kk - acc; break; }
            acc += h8[b];
          }
        }
      }
      __syncthreads();
    }
    T = sh[0];
    k_eq = sh[1];
  }
  __syncthreads();
  // ordered compaction over [0, m): one contiguous chunk per warp
  const int chunk = (((m + NW - 1) / NW) + 31) / 32 * 32;
  const int lo = warp * chunk, hi = min(m, lo + chunk);
  unsigned int gt = 0, eq = 0;
  for (int base = lo; base < hi; base += 32) {
    const int i = base + lane;
    const bool in = i < hi;
    const uint32_t key = in ? f32_order_key(score[i]) : 0u;
    gt += __popc(__ballot_sync(0xffffffffu, in && take > 0 && key > T));
    eq += __popc(__ballot_sync(0xffffffffu, in && take > 0 && key == T));
  }
  if (lane == 0) { wcnt[warp] = gt; wcnt[NW + warp] = eq; }
  __syncthreads();
  unsigned int gt_before = 0, eq_before = 0;
  for (int w = 0; w < warp; ++w) { gt_before += wcnt[w]; eq_before += wcnt[NW + w]; }
  unsigned int pos = gt_before + min(k_eq, eq_before), eq_run = eq_before;
  const unsigned int lt_mask = (1u << lane) - 1u;
  for (int base = lo; base < hi; base += 32) {
    const int i = base + lane;
    const bool in = i < hi && take > 0;
    const uint32_t key = in ? f32_order_key(score[i]) : 0u;
    const bool is_eq = in && key == T;
    const unsigned int beq = __ballot_sync(0xffffffffu, is_eq);
    const bool tk = in && (key > T || (is_eq && eq_run + __popc(beq & lt_mask) < k_eq));
    const unsigned int bt = __ballot_sync(0xffffffffu, tk);
    if (tk) {
      const unsigned int p = pos + __popc(bt & lt_mask);
      if ((int)p < cap) out[p] = i;
    }
    pos += __popc(bt);
    eq_run += __popc(beq);
  }
  if (tid == 0 && take < cap) out[take] = qb;     // the diagonal block is the largest index: list stays ascending
  __syncthreads();
  return take + 1;
}

// k is read as 16-byte vectors (rows of the pooled arrays are 512-byte aligned); the products are still accumulated
// one after the other in the order t = 0..127, so every kernel that calls this gets the same bits.
__device__ __forceinline__ float pooled_score(const float* q, const float* k, float scale) {
  float acc = 0.f;
  const float4* k4 = reinterpret_cast<const float4*>(k);
#pragma unroll 4
  for (int t = 0; t < RS_HEAD_DIM / 4; ++t) {
    const float4 kv = k4[t];
    acc = fmaf(q[4 * t], kv.x, acc);
    acc = fmaf(q[4 * t + 1], kv.y, acc);
    acc = fmaf(q[4 * t + 2], kv.z, acc);
    acc = fmaf(q[4 * t + 3], kv.w, acc);
  }
  return acc * scale;
}

// Pooled scores of the last query block of an item that has a block-sparse candidate to evaluate: 256 key blocks
// per thread block.
__device__ __forceinline__ void bs_eval_scores_block(const IdxParams& P, int item, int bx) {
  __shared__ float qrow[RS_HEAD_DIM];
  const int s = item / P.Hq, h = item - s * P.Hq, g = h / P.group;
  const int qb = (P.seg_bounds[s + 1] >> 6) - 1;
  if (bx * 256 >= qb) return;
  if (threadIdx.x < RS_HEAD_DIM) qrow[threadIdx.x] = P.qpool[((size_t)h * P.nb + qb) * RS_HEAD_DIM + threadIdx.x];
  __syncthreads();
  const int kb = bx * 256 + threadIdx.x;
  if (kb < qb)
    P.bs_eval_ws[(size_t)item * P.nb + kb] = pooled_score(qrow, P.kpool + ((size_t)g * P.nb + kb) * RS_HEAD_DIM, P.scale);
}

// Evaluation of one block-sparse candidate of one item: the candidate's selection from the pooled scores of the
// segment's last query block (list, coverage, pairs).  bs_index counts the library's block-sparse candidates.
// All kFinishThreads threads of the block call it.
__device__ __forceinline__ void bs_eval_block(const IdxParams& P, int item, int bs_index, float* score /* [nb] */) {
  constexpr int NT = kFinishThreads;
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sh[8];
  __shared__ unsigned int wcnt[2 * NT / 32];
  __shared__ int32_t sel[1024];
  __shared__ u64 cov[RS_PROBE_GROUPS];
  if (P.stats == nullptr && P.choice != nullptr) return;    // materialise mode without stats: rows are built elsewhere
  int my_c = -1;
  for (int c = 0, seen = 0; c < P.n_cand; ++c)
    if (P.lib[c].pattern == RS_BLOCK_SPARSE && seen++ == bs_index) my_c = c;
  if (my_c < 0 || (P.choice != nullptr && P.choice[item] != my_c)) return;
  const int s = item / P.Hq;
  const int q0 = P.seg_bounds[s], q1 = P.seg_bounds[s + 1];
  const int qb = (q1 >> 6) - 1;
  const int tid = threadIdx.x;
  if (P.bscore != nullptr) {
    const float* row = P.bscore + ((size_t)item * P.nb + qb) * P.nb;
    for (int kb = tid; kb < qb; kb += NT) score[kb] = row[kb];
  } else {
    const float* row = P.bs_eval_ws + (size_t)item * P.nb;
    for (int kb = tid; kb < qb; kb += NT) score[kb] = row[kb];
  }
  __syncthreads();
  {
    const int c = my_c;
    const rs_candidate cand = P.lib[c];
    const int slot = (P.choice != nullptr) ? item : item * P.n_cand + c;
    if (tid < RS_PROBE_GROUPS) cov[tid] = 0;
    __syncthreads();
    const int k_b = min(cand.b0, 1024);
    const int cnt = select_row<NT>(score, qb, min(k_b, qb + 1) - 1, qb, sel, 1024, hist, sh, wcnt);
    if (P.choice == nullptr) {
      int32_t* dst = P.out.bs_blk + (size_t)slot * P.out.kb_cap;
      for (int i = tid; i < cnt && i < P.out.kb_cap; i += NT) dst[i] = sel[i];
      if (tid == 0) P.out.bs_count[slot] = cnt;
    }
    if (P.stats != nullptr) {
      const u64* vblk = P.vblk + (size_t)item * RS_PROBE_GROUPS * P.nb;
      u64 part[RS_PROBE_GROUPS] = {0, 0, 0, 0};
      for (int i = tid; i < cnt; i += NT)
#pragma unroll
        for (int gg = 0; gg < RS_PROBE_GROUPS; ++gg) part[gg] += vblk[(size_t)gg * P.nb + sel[i]];
#pragma unroll
      for (int gg = 0; gg < RS_PROBE_GROUPS; ++gg) warp_sum_then_add(part[gg], &cov[gg]);
      __syncthreads();
      if (tid == 0) {
        rs_cand_stats* st = P.stats + (size_t)item * P.n_cand + c;
        for (int gg = 0; gg < RS_PROBE_GROUPS; ++gg) st->cov_fx[gg] = cov[gg];
        st->pairs = pairs_block_sparse(q0 >> 6, q1 >> 6, cand.b0);
      }
    }
    __syncthreads();
  }
}

// What follows the line selection, one kernel: blocks 0 .. n_finish - 1 turn the selected lines of a vertical-slash
// job into D, coverage and pairs (job = block); the blocks behind them evaluate one (item, block-sparse candidate) each.
__global__ void __launch_bounds__(kFinishThreads)
rs_finish_eval_kernel(IdxParams P, int n_finish, int n_items) {
  extern __shared__ float score[];      // [nb], used by the block-sparse part
  if ((int)blockIdx.x < n_finish) {
    vs_finish_block(P, blockIdx.x);
  } else {
    const int e = blockIdx.x - n_finish;
    bs_eval_block(P, e % n_items, e / n_items, score);
  }
}

// What the side chain starts with, one kernel: blocks 0 .. n_simple - 1 the statistics of the closed-form candidates
// (job = block), the blocks behind them the pooled scores the block-sparse evaluation selects from (score_blocks
// blocks per item).
__global__ void __launch_bounds__(256)
rs_side_stats_kernel(IdxParams P, int n_simple, int score_blocks) {
  if ((int)blockIdx.x < n_simple) {
    simple_stats_block(P, blockIdx.x);
  } else {
    const int e = blockIdx.x - n_simple;
    bs_eval_scores_block(P, e / score_blocks, e % score_blocks);
  }
}

// Materialise: one block per (query block, head) of every item routed to block-sparse.
__device__ __forceinline__ void bs_row_block(const IdxParams& P, int qb, int h, float* score /* [nb] */) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sh[8];
  __shared__ unsigned int wcnt[16];
  const int s = seg_of_block(P, qb);
  const int item = s * P.Hq + h;
  const rs_candidate cand = P.lib[P.choice[item]];
  if (cand.pattern != RS_BLOCK_SPARSE) return;
  const int tid = threadIdx.x;
  const float* row = (P.bscore != nullptr) ? P.bscore + ((size_t)item * P.nb + qb) * P.nb
                                           : P.bs_ws + ((size_t)h * P.nb + qb) * P.nb;
  for (int kb = tid; kb < qb; kb += 256) score[kb] = row[kb];
  __syncthreads();
  const size_t orow = (size_t)h * P.nb + qb;
  const int k_b = min(cand.b0, P.out.kb_cap);
  const int cnt = select_row<256>(score, qb, min(k_b, qb + 1) - 1, qb, P.out.bs_blk + orow * P.out.kb_cap, P.out.kb_cap,
                                  hist, sh, wcnt);
  if (tid == 0) P.out.bs_count[orow] = cnt;
}

// The same selection for query blocks with at most 1024 candidate key blocks, one warp per query block: every lane
// keeps its strided share of the row's ranking keys in registers, the take-th largest key is built bit by bit from
// the top (a count over the row per bit), then an ordered compaction by ballots writes the ascending list.  Same
// order as select_row (key descending, index ascending), without block-wide barriers.
constexpr int kWarpRowMax = 1024;

__device__ __forceinline__ void bs_row_warp(const IdxParams& P, int qb, int h) {
  const int lane = threadIdx.x & 31;
  const int s = seg_of_block(P, qb);
  const int item = s * P.Hq + h;
  const rs_candidate cand = P.lib[P.choice[item]];
  if (cand.pattern != RS_BLOCK_SPARSE) return;
  const float* row = (P.bscore != nullptr) ? P.bscore + ((size_t)item * P.nb + qb) * P.nb
                                           : P.bs_ws + ((size_t)h * P.nb + qb) * P.nb;
  const int m = qb;                                   // candidates: key blocks 0 .. qb - 1
  const size_t orow = (size_t)h * P.nb + qb;
  int32_t* out = P.out.bs_blk + orow * P.out.kb_cap;
  const int cap = P.out.kb_cap;
  const int take = min(min(min(cand.b0, cap), qb + 1) - 1, m);
  uint32_t key[kWarpRowMax / 32];
#pragma unroll
  for (int c = 0; c < kWarpRowMax / 32; ++c) {
    const int i = c * 32 + lane;
    key[c] = (i < m) ? f32_order_key(row[i]) : 0u;    // finite scores have keys > 0: the padding is never counted
  }
  uint32_t T = 0u;
  int k_eq = 0;
  if (take > 0) {
    for (int b = 31; b >= 0; --b) {
      const uint32_t Tc = T | (1u << b);
      int cnt = 0;
#pragma unroll
      for (int c = 0; c < kWarpRowMax / 32; ++c)
        if (c * 32 < m) cnt += (key[c] >= Tc) ? 1 : 0;
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (cnt >= take) T = Tc;
    }
    int gt = 0;
#pragma unroll
    for (int c = 0; c < kWarpRowMax / 32; ++c)
      if (c * 32 < m) gt += (key[c] > T) ? 1 : 0;
    k_eq = take - __reduce_add_sync(0xffffffffu, gt);
  }
  const unsigned int lt_mask = (1u << lane) - 1u;
  int pos = 0, eq_run = 0;
#pragma unroll
  for (int c = 0; c < kWarpRowMax / 32; ++c) {
    if (c * 32 < m && take > 0) {
      const int i = c * 32 + lane;
      const bool in = i < m;
      const bool is_eq = in && key[c] == T;
      const unsigned int beq = __ballot_sync(0xffffffffu, is_eq);
      const bool tk = in && (key[c] > T || (is_eq && eq_run + __popc(beq & lt_mask) < k_eq));
      const unsigned int bt = __ballot_sync(0xffffffffu, tk);
      if (tk) {
        const int p = pos + __popc(bt & lt_mask);
        if (p < cap) out[p] = i;
      }
      pos += __popc(bt);
      eq_run += __popc(beq);
    }
  }
  if (lane == 0) {
    if (take < cap) out[take] = qb;                   // the diagonal block is the largest index: list stays ascending
    P.out.bs_count[orow] = take + 1;
  }
}

// Row selection of the materialise call, one kernel: blocks 0 .. ceil(n_short / 8) - 1 serve the query blocks below
// n_short one warp each, the blocks behind them one longer row each.
__global__ void __launch_bounds__(256)
rs_bs_rows_kernel(IdxParams P, int n_short) {
  extern __shared__ float score[];      // [nb], used by the block-per-row part
  const int n_warp_blocks = (n_short + 7) / 8;
  const int h = blockIdx.y;
  if ((int)blockIdx.x < n_warp_blocks) {
    const int qb = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (qb < n_short) bs_row_warp(P, qb, h);
  } else {
    bs_row_block(P, n_short + ((int)blockIdx.x - n_warp_blocks), h, score);
  }
}

// Fused pooled scores for the items routed to block-sparse: 64 x 64 tiles of qpool[h] kpool[g]^T / sqrt(d),
// lower triangle only; every output accumulates k = 0..127 in order with fmaf (same bits as pooled_score).
__global__ void __launch_bounds__(256)
rs_bs_scores_kernel(IdxParams P) {
  __shared__ float As[64][33], Bs[64][33];
  __shared__ int any_bs;
  const int kt = blockIdx.x, qt = blockIdx.y, h = blockIdx.z;
  if (kt > qt) return;
  const int tid = threadIdx.x;
  if (tid == 0) any_bs = 0;
  __syncthreads();
  if (tid < 64) {
    const int qb = qt * 64 + tid;
    if (qb < P.nb) {
      const int item = seg_of_block(P, qb) * P.Hq + h;
      if (P.lib[P.choice[item]].pattern == RS_BLOCK_SPARSE) any_bs = 1;
    }
  }
  __syncthreads();
  if (!any_bs) return;
  const int g = h / P.group;
  const int tx = tid & 15, ty = tid >> 4;       // outputs rows ty*4.., cols tx*4..
  float acc[4][4] = {};
  for (int k0 = 0; k0 < RS_HEAD_DIM; k0 += 32) {
    for (int i = tid; i < 64 * 32; i += 256) {
      const int r = i >> 5, cidx = i & 31;
      const int qb = qt * 64 + r, kb = kt * 64 + r;
      As[r][cidx] = (qb < P.nb) ? P.qpool[((size_t)h * P.nb + qb) * RS_HEAD_DIM + k0 + cidx] : 0.f;
      Bs[r][cidx] = (kb < P.nb) ? P.kpool[((size_t)g * P.nb + kb) * RS_HEAD_DIM + k0 + cidx] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < 32; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[ty * 4 + i][k]; b[i] = Bs[tx * 4 + i][k]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int qb = qt * 64 + ty * 4 + i;
    if (qb >= P.nb) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int kb = kt * 64 + tx * 4 + j;
      if (kb < P.nb) P.bs_ws[((size_t)h * P.nb + qb) * P.nb + kb] = acc[i][j] * P.scale;
    }
  }
}

// ------------------------------------------------------------------------------------------ mixture coverage
// Coverage of every candidate's mask on the rows of the query mixture (Section 3.2, Eq. 4: "u measures disagreement
// among probe subsets").  The pooled probe resolves key blocks of 64, so the mass of a block is split evenly over its
// visible keys: row i of candidate c collects  sum_kb  fx(A[i][kb]) * num_c(i, kb) / den(i, kb)  with den the number of
// visible keys of the block (j <= i) and num how many of them the candidate's mask row selects; integer arithmetic, so
// the sums do not depend on the order of evaluation.  One block per (probe row, item); candidates in a loop.
struct MixArgs {
  const float* A;          // [n_seg][Hq][r][nb] probabilities of the pooled probe at g = 64
  const int32_t* rows;     // [n_seg][r]
  int r, n_sub;
  int sub_bounds[5];
  u64* covmix;             // [n_items][n_cand][4]
};

__device__ __forceinline__ int interval_len(int lo, int hi) { return hi >= lo ? hi - lo + 1 : 0; }

constexpr int kMixMaxVS = 4, kMixMaxBS = 4;      // vertical-slash / block-sparse candidates per library served here

// One block per run of consecutive mixture rows that share a query block and a subset (the recent rows, the
// boundary rows, every uniform row); the other blocks of the grid leave at once.  Prologue: per vertical-slash
// candidate the block-diagonal bitmap and the number of selected columns per key block, per block-sparse candidate the
// membership bitmap of the query block's selection.  Then one sweep over (row, key block) feeds all candidates.
__global__ void __launch_bounds__(256)
rs_mix_cov_kernel(IdxParams P, MixArgs M) {
  extern __shared__ float mix_smem[];
  // score[nb] | blist[kb_cap] | vcnt[kMixMaxVS][nb] | dbits[kMixMaxVS][128] | member[kMixMaxBS][nb / 32 + 1] | diagcols[kMixMaxVS][64]
  float* score = mix_smem;
  int32_t* blist = reinterpret_cast<int32_t*>(score + P.nb);
  int* vcnt = reinterpret_cast<int*>(blist + P.out.kb_cap);
  uint32_t* dbits = reinterpret_cast<uint32_t*>(vcnt + kMixMaxVS * P.nb);
  const int mw = P.nb / 32 + 1;
  uint32_t* member = dbits + kMixMaxVS * 128;
  int* diagcols = reinterpret_cast<int*>(member + kMixMaxBS * mw);
  __shared__ int n_diagcols[kMixMaxVS];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sh[8];
  __shared__ unsigned int wcnt[16];
  __shared__ u64 red[8];
  __shared__ float qrow[RS_HEAD_DIM];
  const int t0 = blockIdx.x, item = blockIdx.y;
  const int s = item / P.Hq, h = item - s * P.Hq, g = h / P.group;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* rows = M.rows + s * M.r;
  int sub = 0;
  while (sub + 1 < M.n_sub && t0 >= M.sub_bounds[sub + 1]) ++sub;
  const int qb_i = rows[t0] >> 6;
  if (t0 > M.sub_bounds[sub] && (rows[t0 - 1] >> 6) == qb_i) return;      // not the first row of its run
  int t1 = t0 + 1;
  while (t1 < M.sub_bounds[sub + 1] && (rows[t1] >> 6) == qb_i) ++t1;
  // a long run (the 32 recent rows) is shared by the blocks of grid.z: block z takes rows t0 + z, t0 + z + gridDim.z, ..
  if (t0 + (int)blockIdx.z >= t1) return;

  // ---- prologue
  int vs_of[kMixMaxVS], bs_of[kMixMaxBS];
  int n_vs = 0, n_bs = 0;
  for (int c = 0; c < P.n_cand; ++c) {
    if (P.lib[c].pattern == RS_VERTICAL_SLASH && n_vs < kMixMaxVS) {
#pragma unroll
      for (int e = 0; e < kMixMaxVS; ++e) if (e == n_vs) vs_of[e] = c;
      ++n_vs;
    }
    if (P.lib[c].pattern == RS_BLOCK_SPARSE && n_bs < kMixMaxBS) {
#pragma unroll
      for (int e = 0; e < kMixMaxBS; ++e) if (e == n_bs) bs_of[e] = c;
      ++n_bs;
    }
  }
  for (int x = tid; x < kMixMaxVS * P.nb; x += 256) vcnt[x] = 0;
  for (int x = tid; x < kMixMaxVS * 128; x += 256) dbits[x] = 0;
  for (int x = tid; x < kMixMaxBS * mw; x += 256) member[x] = 0;
  if (tid < kMixMaxVS) n_diagcols[tid] = 0;
  __syncthreads();
#pragma unroll
  for (int v = 0; v < kMixMaxVS; ++v) {
    if (v >= n_vs) continue;
    const int slot = item * P.n_cand + vs_of[v];
    const int n_cols = P.out.vs_count[4 * slot + 0], n_diag = P.out.vs_count[4 * slot + 2];
    const int32_t* cols = P.out.vs_cols + (size_t)slot * P.out.kv_cap;
    const int32_t* diag = P.out.vs_diag + (size_t)slot * P.out.nd_cap;
    for (int x = tid; x < n_diag; x += 256) { const int d = diag[x]; atomicOr(&dbits[v * 128 + (d >> 5)], 1u << (d & 31)); }
    for (int x = tid; x < n_cols; x += 256) {
      const int j = cols[x];
      const int kb = j >> 6;
      if (kb < qb_i) atomicAdd(&vcnt[v * P.nb + kb], 1);
      else if (kb == qb_i) { const int at = atomicAdd(&n_diagcols[v], 1); diagcols[v * 64 + at] = j; }   // tested per row
    }
  }
  if (n_bs > 0 && qb_i == (P.seg_bounds[s + 1] >> 6) - 1) {
    // the segment's last query block: the evaluation already selected for it (evaluation layout, slot = item, candidate)
#pragma unroll
    for (int b = 0; b < kMixMaxBS; ++b) {
      if (b >= n_bs) continue;
      const size_t slot = (size_t)item * P.n_cand + bs_of[b];
      const int cnt = P.out.bs_count[slot];
      const int32_t* bl = P.out.bs_blk + slot * P.out.kb_cap;
      for (int x = tid; x < cnt; x += 256) { const int kb = bl[x]; atomicOr(&member[b * mw + (kb >> 5)], 1u << (kb & 31)); }
    }
  } else if (n_bs > 0) {
    if (tid < RS_HEAD_DIM) qrow[tid] = P.qpool[((size_t)h * P.nb + qb_i) * RS_HEAD_DIM + tid];
    __syncthreads();
    for (int kb = tid; kb < qb_i; kb += 256)
      score[kb] = pooled_score(qrow, P.kpool + ((size_t)g * P.nb + kb) * RS_HEAD_DIM, P.scale);
    __syncthreads();
#pragma unroll
    for (int b = 0; b < kMixMaxBS; ++b) {
      if (b >= n_bs) continue;
      const int k_b = min(P.lib[bs_of[b]].b0, P.out.kb_cap);
      const int cnt = select_row<256>(score, qb_i, min(k_b, qb_i + 1) - 1, qb_i, blist, P.out.kb_cap, hist, sh, wcnt);
      for (int x = tid; x < cnt; x += 256) { const int kb = blist[x]; atomicOr(&member[b * mw + (kb >> 5)], 1u << (kb & 31)); }
      __syncthreads();
    }
  }
  __syncthreads();

  // ---- one sweep over (row, key block) for all candidates
  u64 part[RS_MAX_CANDIDATES];
#pragma unroll
  for (int c = 0; c < RS_MAX_CANDIDATES; ++c) part[c] = 0;
  for (int t = t0 + (int)blockIdx.z; t < t1; t += (int)gridDim.z) {
    const int i = rows[t];
    const float* a = M.A + (((size_t)s * P.Hq + h) * M.r + t) * (size_t)P.nb;
    for (int kb = tid; kb <= qb_i; kb += 256) {
      const u64 af = fx(a[kb]);
      if (af == 0) continue;
      const int lo = kb * 64, hi = min(lo + 63, i);
      const u64 den = (u64)(hi - lo + 1);
      int iv = 0, ib = 0;
#pragma unroll
      for (int c = 0; c < RS_MAX_CANDIDATES; ++c) {
        if (c >= P.n_cand) continue;
        const rs_candidate cand = P.lib[c];
        u64 num;
        if (cand.pattern == RS_DENSE) {
          num = den;
        } else if (cand.pattern == RS_A_SHAPE) {
          const int s_hi = min(hi, cand.b0 - 1), w_lo = max(lo, i - cand.b1 + 1);
          num = (u64)(interval_len(lo, s_hi) + interval_len(w_lo, hi) - interval_len(w_lo, s_hi));
        } else if (cand.pattern == RS_VERTICAL_SLASH) {
          const int v = iv++;
          if (v >= kMixMaxVS) { num = 0; }
          else {
            const int d = qb_i - kb;
            if ((dbits[v * 128 + (d >> 5)] >> (d & 31)) & 1u) num = den;
            else if (kb < qb_i) num = (u64)vcnt[v * P.nb + kb];
            else {
              int cntd = 0;
              for (int x = 0; x < n_diagcols[v]; ++x) cntd += (diagcols[v * 64 + x] <= i);
              num = (u64)cntd;
            }
          }
        } else {
          const int b = ib++;
          num = (b < kMixMaxBS && ((member[b * mw + (kb >> 5)] >> (kb & 31)) & 1u)) ? den : 0;
        }
        part[c] += (den == 64) ? ((af * num) >> 6) : (af * num / den);      // 64-bit division only on the row's own block
      }
    }
  }
#pragma unroll
  for (int c = 0; c < RS_MAX_CANDIDATES; ++c) {
    if (c >= P.n_cand) continue;
    u64 v = part[c];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (tid == 0) {
      u64 tot = 0;
      for (int w8 = 0; w8 < 8; ++w8) tot += red[w8];
      atomicAdd(&M.covmix[((size_t)item * P.n_cand + c) * 4 + sub], tot);
    }
  }
}

struct IdxPlan { size_t vblk, bs_ws, keys, bs_eval, total; };

IdxPlan plan(const rs_problem* p, const rs_candidate* lib, int n_cand) {
  IdxPlan w{};
  const size_t nb = (size_t)p->n_keys / 64;
  const size_t items = (size_t)p->n_segments * p->n_q_heads;
  bool any_bs = false, any_vs = false;
  for (int c = 0; c < n_cand; ++c) { any_bs |= (lib[c].pattern == RS_BLOCK_SPARSE); any_vs |= (lib[c].pattern == RS_VERTICAL_SLASH); }
  size_t off = 0;
  w.vblk = off;  off += rs_align_up(items * RS_PROBE_GROUPS * nb * sizeof(u64), 256);
  w.bs_ws = off; off += any_bs ? rs_align_up((size_t)p->n_q_heads * nb * nb * sizeof(float), 256) : 0;
  w.keys = off;  off += any_vs ? rs_align_up(items * 2 * (size_t)p->n_keys * sizeof(u64), 256) : 0;
  w.bs_eval = off; off += any_bs ? rs_align_up(items * nb * sizeof(float), 256) : 0;
  w.total = off;
  return w;
}

}  // namespace

size_t rs_indices_workspace_bytes(const rs_problem* p, const rs_candidate* lib, int n_cand) {
  return plan(p, lib, n_cand).total;
}

static int build_indices_impl(const rs_problem* p, const rs_candidate* lib, int n_cand, const float* vert,
                              const float* slash, const float* rank_vert, const float* rank_slash, const float* qpool,
                              const float* kpool, const float* bscore, const int32_t* choice, const rs_index_set* out,
                              rs_cand_stats* stats, void* ws, size_t ws_bytes, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!lib || n_cand <= 0 || n_cand > RS_MAX_CANDIDATES || !out || !ws) return RS_ERR_INVALID_ARG;
  if (choice == nullptr && stats == nullptr) return RS_ERR_INVALID_ARG;
  const int n_items = p->n_segments * p->n_q_heads;
  const int nb = p->n_keys / 64;
  bool any_vs = false, any_bs = false;
  for (int c = 0; c < n_cand; ++c) {
    const rs_candidate& cd = lib[c];
    if (cd.pattern < 0 || cd.pattern > 3) return RS_ERR_INVALID_ARG;
    if (cd.pattern == RS_VERTICAL_SLASH) {
      any_vs = true;
      if (cd.b0 < 0 || cd.b1 < 1) return RS_ERR_INVALID_ARG;
      if (out->kv_cap < (cd.b0 < p->n_keys ? cd.b0 : p->n_keys) || out->ks_cap < (cd.b1 < p->n_keys ? cd.b1 : p->n_keys) ||
          out->nd_cap < nb) return RS_ERR_INVALID_ARG;
    } else if (cd.pattern == RS_BLOCK_SPARSE) {
      any_bs = true;
      if (cd.b0 < 1 || cd.b0 > 1024) return RS_ERR_INVALID_ARG;
      if (out->kb_cap < (cd.b0 < nb ? cd.b0 : nb)) return RS_ERR_INVALID_ARG;
    } else if (cd.pattern == RS_A_SHAPE) {
      if (cd.b0 < 0 || cd.b1 < 1) return RS_ERR_INVALID_ARG;
      if (stats != nullptr) {
        // coverage of sink + window from column and offset masses needs the two not to overlap on the probe rows
        for (int s = 0; s < p->n_segments; ++s) {
          const int q1 = p->seg_bounds[s + 1];
          if (cd.b1 < q1 && q1 - RS_PROBE_ROWS - cd.b1 + 1 < cd.b0) return RS_ERR_UNSUPPORTED_SHAPE;
        }
      }
    }
  }
  if ((any_vs || stats) && (!vert || !slash)) return RS_ERR_INVALID_ARG;
  if (any_bs && bscore == nullptr && (!qpool || !kpool)) return RS_ERR_INVALID_ARG;
  const int n_slots = choice ? n_items : n_items * n_cand;
  // materialise mode with n_vs_slots == 0: the caller keeps using the lists of an earlier evaluation call
  const bool skip_vs = choice != nullptr && out->n_vs_slots == 0 && stats == nullptr;
  if (any_vs && !skip_vs && out->n_vs_slots < n_slots) return RS_ERR_INVALID_ARG;
  if (any_bs && out->bs_rows < (choice ? p->n_q_heads * nb : n_slots)) return RS_ERR_INVALID_ARG;
  for (int s = 0; s < p->n_segments; ++s)
    if (p->seg_bounds[s + 1] < RS_PROBE_ROWS) return RS_ERR_UNSUPPORTED_SHAPE;
  const IdxPlan w = plan(p, lib, n_cand);
  if (ws_bytes < w.total) return RS_ERR_WORKSPACE_TOO_SMALL;
  if (((uintptr_t)ws & 255) != 0) return RS_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);

  IdxParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = P.Hq / P.Hkv; P.n_seg = p->n_segments;
  P.n_cand = n_cand; P.nb = nb;
  for (int s = 0; s <= p->n_segments; ++s) P.seg_bounds[s] = p->seg_bounds[s];
  for (int c = 0; c < n_cand; ++c) P.lib[c] = lib[c];
  P.vert = vert; P.slash = slash; P.qpool = qpool; P.kpool = kpool; P.bscore = bscore; P.choice = choice;
  P.rank_vert = rank_vert ? rank_vert : vert; P.rank_slash = rank_slash ? rank_slash : slash;
  P.out = *out; P.stats = stats; P.vblk = reinterpret_cast<u64*>(wsb + w.vblk);
  P.bs_ws = reinterpret_cast<float*>(wsb + w.bs_ws); P.status = status;
  P.keys = reinterpret_cast<u64*>(wsb + w.keys);
  P.bs_eval_ws = reinterpret_cast<float*>(wsb + w.bs_eval);
  P.scale = (float)(1.0 / sqrt((double)RS_HEAD_DIM));

  const int n_jobs = n_items * n_cand;
  // the ranking-key kernel also writes the block sums of fx(vert) when the lists are ranked by vert itself
  const bool fuse_vblk = stats != nullptr && any_vs && P.rank_vert == vert;
  if (stats != nullptr && !fuse_vblk) {
    const long long warps = (long long)n_items * RS_PROBE_GROUPS * nb;
    rs_vblk_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, stream>>>(P);
  }
  // The line selection of the vertical-slash candidates on one side, the closed-form statistics, the pooled scores and
  // the materialised block-sparse rows on the other do not read each other's results; the second group runs on the
  // side stream.  What comes after the selection (D / coverage / pairs, and the block-sparse evaluation, which reads
  // the pooled scores) is one kernel behind the join.
  // launch shape of the select kernel; its attribute is set before the fork so that no error path sits between the
  // fork and the join below
  int n_vs = 0, n_bs = 0;
  for (int c = 0; c < n_cand; ++c) { n_vs += (lib[c].pattern == RS_VERTICAL_SLASH); n_bs += (lib[c].pattern == RS_BLOCK_SPARSE); }
  const int sel_groups = choice ? 1 : (n_vs + kSelMaxC - 1) / kSelMaxC;
  const size_t sel_smem = (size_t)(choice ? 1 : kSelMaxC) * kBins * sizeof(unsigned int);
  static rs_smem_attr sel_attr;
  if (rs_ensure_dynamic_smem(sel_attr, rs_vs_select_kernel, (int)(kSelMaxC * kBins * sizeof(unsigned int))) != RS_OK)
    return RS_ERR_CUDA;
  const bool two_chains = any_vs && !skip_vs && (any_bs || stats != nullptr);
  cudaStream_t side = stream;
  // the ranking keys (and with them the block sums both chains read) come before the fork
  if (any_vs && !skip_vs) rs_vs_keys_kernel<<<dim3((P.n + 255) / 256, 2 * n_items), 256, 0, stream>>>(P, fuse_vblk ? 1 : 0);
  if (two_chains) {
    rc = rs_side_fork(stream, &side);
    if (rc != RS_OK) return rc;
  }
  if (any_vs && !skip_vs) rs_vs_select_kernel<<<dim3(kSelCluster, 2 * n_items, sel_groups), kSelThreads, sel_smem, stream>>>(P);
  const bool eval = any_bs && (choice == nullptr || stats != nullptr);
  {
    const int n_simple = stats != nullptr ? n_jobs : 0;
    const int score_blocks = eval && bscore == nullptr ? (nb + 255) / 256 : 0;
    if (n_simple + score_blocks > 0)
      rs_side_stats_kernel<<<n_simple + score_blocks * n_items, 256, 0, side>>>(P, n_simple, score_blocks);
  }
  if (any_bs && choice != nullptr) {
    if (bscore == nullptr) {
      const int nt = (nb + 63) / 64;
      rs_bs_scores_kernel<<<dim3(nt, nt, P.Hq), 256, 0, side>>>(P);
    }
    // short rows one warp each; rows with more than 1024 candidate blocks one thread block each
    const int n_short = nb < kWarpRowMax + 1 ? nb : kWarpRowMax + 1;       // query blocks 0 .. 1024
    rs_bs_rows_kernel<<<dim3((n_short + 7) / 8 + (nb - n_short), P.Hq), 256, (size_t)nb * sizeof(float), side>>>(P, n_short);
  }
  if (two_chains) {
    rc = rs_side_join(stream);
    if (rc != RS_OK) return rc;
  }
  // after the line selection (and, for the block-sparse evaluation, the pooled scores of the side chain)
  {
    const int n_finish = any_vs && !skip_vs ? n_jobs : 0;
    const int n_eval = eval ? n_items * n_bs : 0;
    if (n_finish + n_eval > 0)
      rs_finish_eval_kernel<<<n_finish + n_eval, kFinishThreads, (size_t)nb * sizeof(float), stream>>>(P, n_finish, n_items);
  }
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

extern "C" int rs_build_indices(const rs_problem* p, const rs_candidate* lib, int n_cand, const float* vert,
                                const float* slash, const float* qpool, const float* kpool, const float* bscore,
                                const int32_t* choice, const rs_index_set* out, rs_cand_stats* stats, void* ws,
                                size_t ws_bytes, int32_t* status, void* stream) {
  return build_indices_impl(p, lib, n_cand, vert, slash, nullptr, nullptr, qpool, kpool, bscore, choice, out, stats, ws,
                            ws_bytes, status, stream);
}

extern "C" int rs_build_indices_ranked(const rs_problem* p, const rs_candidate* lib, int n_cand, const float* vert,
                                       const float* slash, const float* rank_vert, const float* rank_slash,
                                       const float* qpool, const float* kpool, const float* bscore, const int32_t* choice,
                                       const rs_index_set* out, rs_cand_stats* stats, void* ws, size_t ws_bytes,
                                       int32_t* status, void* stream) {
  if (!rank_vert || !rank_slash) return RS_ERR_INVALID_ARG;
  return build_indices_impl(p, lib, n_cand, vert, slash, rank_vert, rank_slash, qpool, kpool, bscore, choice, out, stats,
                            ws, ws_bytes, status, stream);
}

extern "C" int rs_mixture_coverage(const rs_problem* p, const rs_candidate* lib, int n_cand, const float* A,
                                   const int32_t* rows, int r, const int32_t* sub_bounds, int n_sub,
                                   const rs_index_set* idx_eval, const float* qpool, const float* kpool,
                                   uint64_t* covmix, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!lib || n_cand <= 0 || n_cand > RS_MAX_CANDIDATES || !A || !rows || !sub_bounds || !idx_eval || !covmix)
    return RS_ERR_INVALID_ARG;
  if (r < 1 || r > 64 || n_sub < 1 || n_sub > 4 || sub_bounds[0] != 0 || sub_bounds[n_sub] != r) return RS_ERR_INVALID_ARG;
  const int n_items = p->n_segments * p->n_q_heads;
  const int nb = p->n_keys / 64;
  bool any_vs = false, any_bs = false;
  for (int c = 0; c < n_cand; ++c) {
    any_vs |= lib[c].pattern == RS_VERTICAL_SLASH;
    any_bs |= lib[c].pattern == RS_BLOCK_SPARSE;
  }
  if (any_vs && idx_eval->n_vs_slots < n_items * n_cand) return RS_ERR_INVALID_ARG;   // needs the evaluation layout
  if (any_bs && (!qpool || !kpool)) return RS_ERR_INVALID_ARG;
  rc = rs_check_device();
  if (rc != RS_OK) return rc;
  (void)status;
  cudaStream_t stream = (cudaStream_t)stream_;
  IdxParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = P.Hq / P.Hkv; P.n_seg = p->n_segments;
  P.n_cand = n_cand; P.nb = nb;
  for (int s = 0; s <= p->n_segments; ++s) P.seg_bounds[s] = p->seg_bounds[s];
  for (int c = 0; c < n_cand; ++c) P.lib[c] = lib[c];
  P.qpool = qpool; P.kpool = kpool; P.out = *idx_eval;
  P.scale = (float)(1.0 / sqrt((double)RS_HEAD_DIM));
  MixArgs M{};
  M.A = A; M.rows = rows; M.r = r; M.n_sub = n_sub;
  for (int k = 0; k <= n_sub; ++k) M.sub_bounds[k] = sub_bounds[k];
  M.covmix = reinterpret_cast<u64*>(covmix);
  if (cudaMemsetAsync(covmix, 0, (size_t)n_items * n_cand * 4 * sizeof(uint64_t), stream) != cudaSuccess) return RS_ERR_CUDA;
  int n_vs = 0, n_bs = 0;
  for (int c = 0; c < n_cand; ++c) { n_vs += lib[c].pattern == RS_VERTICAL_SLASH; n_bs += lib[c].pattern == RS_BLOCK_SPARSE; }
  if (n_vs > kMixMaxVS || n_bs > kMixMaxBS) return RS_ERR_UNSUPPORTED_SHAPE;
  const size_t smem = (size_t)nb * 4 + (size_t)idx_eval->kb_cap * 4 + (size_t)kMixMaxVS * nb * 4 + kMixMaxVS * 128 * 4 +
                      (size_t)kMixMaxBS * (nb / 32 + 1) * 4 + kMixMaxVS * 64 * 4;
  static rs_smem_attr mix_attr;
  if (rs_ensure_dynamic_smem(mix_attr, rs_mix_cov_kernel, 64 * 1024) != RS_OK) return RS_ERR_CUDA;
  if (smem > 64 * 1024) return RS_ERR_UNSUPPORTED_SHAPE;
  rs_mix_cov_kernel<<<dim3(r, n_items, 4), 256, smem, stream>>>(P, M);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
