// Routed sparse prefill attention (Section 2.1 masked attention, Section 3.4 step 6) and the dense causal
// kernel of Eq. 1, on tcgen05 tensor cores with TMEM accumulators and TMA-fed shared memory.
//
// One CTA owns one 128-row query tile of one head.  The keys a tile visits are a list of 64-key chunks:
// key blocks of K/V selected by the head's pattern (dense, A-shape, the block diagonals of vertical-slash,
// block-sparse) followed by chunks of gathered vertical columns.  Per chunk:
//   S = Q K^T        tcgen05.mma, A and B from shared memory (K-major, 128-byte swizzle), S in TMEM
//   P = exp2(S - m)  softmax warps: tcgen05.ld, online max / sum in one pass per 64-key chunk (rare chunks are
//                    masked in place first), bf16 P written back over S in TMEM
//   O += P V         tcgen05.mma, A = P from TMEM, B = V from shared memory (MN-major)
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps 2-5 = softmax / correction / epilogue.
// Two CTAs share an SM (256 TMEM columns each) so that one tile's softmax overlaps the other's MMAs.
#include <mutex>

#include "common.cuh"

namespace {

rs_smem_attr g_attn_smem;          // dynamic shared memory opt-in of rs_attn_kernel, per device

constexpr int kThreads = 192;
constexpr int kTileM = 128;
constexpr int kChunk = 64;
constexpr int kTmemCols = 256;
constexpr uint32_t kColS = 0;     // two score buffers (fp32, 64 columns each); bf16 P (32 columns) overwrites a buffer's start
constexpr uint32_t kColO = 128;   // O (fp32, 128 columns)

constexpr int kMaskChunks = 128;   // gathered-column chunks with precomputed keep masks (8192 columns); beyond: per element
constexpr uint32_t F_LO = 1u << 12, F_HI = 1u << 13, F_CAUSAL = 1u << 14, F_EDGE = 1u << 15;

struct AttnParams {
  int n, Hq, Hkv, group, n_seg, n_cand;
  int seg_bounds[RS_MAX_SEGMENTS + 1];
  int tile_base[RS_MAX_SEGMENTS + 1];   // first tile id of each segment within one head
  int tiles_per_head;
  rs_candidate lib[RS_MAX_CANDIDATES];
  const int32_t* choice;      // [n_items] or nullptr (all dense)
  rs_index_set idx;
  int kv_pad;                 // rows per slot of the packed vertical K/V
  int vs_eval_layout;         // 1: vertical-slash lists sit in the evaluation layout, slot = item * n_cand + candidate
  const int2* order;          // [n_work] (item, tile in segment), heavy first
  void* O;
  int o_f32;
  float* lse;
  float* onorm;
  unsigned long long* counters;
  int32_t* status;
  float scale_log2e;
};

struct SmemLayout {   // offsets from the 1024-aligned base
  static constexpr uint32_t q = 0, k = 32768, v = 65536, end_tiles = 98304;
};

__device__ __forceinline__ uint32_t range_mask(int lo, int hi, int w) {
  int a = max(lo, 32 * w), b = min(hi, 32 * w + 31);
  if (a > b) return 0u;
  uint32_t len = (uint32_t)(b - a + 1);
  uint32_t m = (len == 32u) ? 0xffffffffu : ((1u << len) - 1u);
  return m << (a - 32 * w);
}

// Masks one 64-key chunk of a score row in place in TMEM (rare chunks only: the causal diagonal, A-shape edges,
// chunks another quarter wants, gathered vertical columns).  Kept out of line so that the common, unmasked chunk
// pays one uniform branch and nothing else.
//   mode 0: every column to -inf;  mode 1: keep j <= i (and, with `edge`, j < n_sink or i - j < window);
//   mode 2: gathered columns: keep vcols[vbase + x] <= i unless a block diagonal of D already covers that key.
//   mode 3: gathered columns with the keep decisions of this row half precomputed per tile: bit x of `keep` says
//           column x survives (valid, not covered by D, not in a later block); bit x of `diag` says the column lies
//           in the row's own key block, where j <= i still has to be tested.
__device__ __noinline__ void rs_mask_chunk(uint32_t taddr, int mode, int i, int j0, int edge, int n_sink, int window,
                                           const int* vcols, int vbase, int n_vcols, const uint32_t* d_bits,
                                           unsigned long long keep = 0ull, unsigned long long diag = 0ull) {
  const uint32_t NEG = 0xff800000u;
  uint32_t x[32];
#pragma unroll 1
  for (int part = 0; part < 2; ++part) {
    tmem_ld32(taddr + 32u * part, x);
    tc_wait_ld();
    const int cb = 32 * part;
    if (mode == 0) {
#pragma unroll
      for (int q = 0; q < 32; ++q) x[q] = NEG;
    } else if (mode == 1) {
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const int j = j0 + cb + q;
        bool keep = j <= i;
        if (edge) keep = keep && (j < n_sink || i - j < window);
        if (!keep) x[q] = NEG;
      }
    } else if (mode == 3) {
      const uint32_t kp = (uint32_t)(keep >> cb), dg = (uint32_t)(diag >> cb);
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (!((kp >> q) & 1u)) x[q] = NEG;
      if (dg != 0u) {
#pragma unroll
        for (int q = 0; q < 32; ++q)
          if (((dg >> q) & 1u) && __ldg(vcols + vbase + cb + q) > i) x[q] = NEG;
      }
    } else {
      const int qb_i = i >> 6;
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const int vi = vbase + cb + q;
        bool keep = false;
        if (vi < n_vcols) {
          const int j = __ldg(vcols + vi);
          if (j <= i) {
            const int dlt = qb_i - (j >> 6);
            keep = !((d_bits[dlt >> 5] >> (dlt & 31)) & 1u);
          }
        }
        if (!keep) x[q] = NEG;
      }
    }
    tmem_st32(taddr + 32u * part, x);
  }
  tc_wait_st();
}

__global__ void __launch_bounds__(kThreads, 2)
rs_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKp,
               const __grid_constant__ CUtensorMap tmVp, const __grid_constant__ AttnParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- work item
  const int2 w = P.order[blockIdx.x];
  const int item = w.x, tile = w.y;
  const int s = item / P.Hq, h = item - s * P.Hq, g = h / P.group;
  const int q0 = P.seg_bounds[s], q1 = P.seg_bounds[s + 1];
  const int i0 = q0 + tile * kTileM;
  const int rows_valid = min(kTileM, q1 - i0);
  const int qb0 = i0 >> 6;
  const bool has_hi = rows_valid > kChunk;
  const int qb_last = has_hi ? qb0 + 1 : qb0;
  const rs_candidate cand = (P.choice != nullptr) ? P.lib[P.choice[item]] : rs_candidate{RS_DENSE, 0, 0, 0};
  const int pattern = cand.pattern;
  const int nb_words = (qb_last >> 5) + 1;

  // ---- shared memory carve-up
  const int list_cap = (P.n >> 6) + 64;
  uint16_t* list = reinterpret_cast<uint16_t*>(sm + SmemLayout::end_tiles);
  uint32_t* lo_bits = reinterpret_cast<uint32_t*>(sm + SmemLayout::end_tiles + ((list_cap * 2 + 15) & ~15));
  uint32_t* hi_bits = lo_bits + 128;
  uint32_t* d_bits = hi_bits + 128;
  int* wprefix = reinterpret_cast<int*>(d_bits + 128);
  uint64_t* bars = reinterpret_cast<uint64_t*>(wprefix + 132);
  volatile int* misc = reinterpret_cast<volatile int*>(bars + 14);   // [0] tmem base, [1] abort, [2] n_block, [3] visible gathered columns
  // keep / own-block masks of the gathered-column chunks: [chunk][row half]
  unsigned long long* vkeep = reinterpret_cast<unsigned long long*>(sm + SmemLayout::end_tiles + ((list_cap * 2 + 15) & ~15) +
                                                                      3 * 128 * 4 + 132 * 4 + 14 * 8 + 64);
  unsigned long long* vdiag = vkeep + 2 * kMaskChunks;
  // barrier pairs (slot 0 / 1) sit next to each other: address of slot s = base + 8 * s
  const uint32_t bar_q = smem_u32(&bars[0]), bar_o = smem_u32(&bars[1]), bar_kf = smem_u32(&bars[2]),
                 bar_ke = smem_u32(&bars[4]), bar_vf = smem_u32(&bars[6]), bar_ve = smem_u32(&bars[8]),
                 bar_s = smem_u32(&bars[10]), bar_p = smem_u32(&bars[12]);
  volatile int* abort_flag = misc + 1;

  if (tid == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_o, 1);
    for (uint32_t sl = 0; sl < 2; ++sl) {
      mbar_init(bar_kf + 8u * sl, 1); mbar_init(bar_ke + 8u * sl, 1); mbar_init(bar_vf + 8u * sl, 1);
      mbar_init(bar_ve + 8u * sl, 1); mbar_init(bar_s + 8u * sl, 1); mbar_init(bar_p + 8u * sl, 128);
    }
    misc[1] = 0; misc[2] = 0; misc[3] = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)&misc[0]), kTmemCols);
    tmem_relinquish();
  }
  for (int i = tid; i < 128; i += kThreads) { lo_bits[i] = 0; hi_bits[i] = 0; d_bits[i] = 0; }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];

  // Q tile load goes out before the chunk list is built.
  if (tid == 0) {
    mbar_arrive_expect_tx(bar_q, 32768);
    tma_load_2d(base + SmemLayout::q, &tmQ, bar_q, 0, h * P.n + i0);
    tma_load_2d(base + SmemLayout::q + 16384, &tmQ, bar_q, 64, h * P.n + i0);
  }

  // ---- chunk list: bitmaps of key blocks wanted by the low / high 64 query rows, then ordered compaction
  int vs_slot = 0, n_vcols = 0;
  if (pattern == RS_VERTICAL_SLASH) {
    vs_slot = P.vs_eval_layout ? item * P.n_cand + P.choice[item] : item;
    const int* cnt = P.idx.vs_count + 4 * vs_slot;
    n_vcols = cnt[0];
    const int n_diag = cnt[2];
    const int* dl = P.idx.vs_diag + (size_t)vs_slot * P.idx.nd_cap;
    for (int i = tid; i < n_diag; i += kThreads) {
      int dlt = dl[i];
      if (dlt >= 0 && dlt < 4096) atomicOr(&d_bits[dlt >> 5], 1u << (dlt & 31));
    }
  } else if (pattern == RS_BLOCK_SPARSE) {
    for (int half = 0; half < (has_hi ? 2 : 1); ++half) {
      const size_t row = (size_t)h * (P.n >> 6) + qb0 + half;
      const int cnt = P.idx.bs_count[row];
      const int* bl = P.idx.bs_blk + row * P.idx.kb_cap;
      uint32_t* dst = half ? hi_bits : lo_bits;
      for (int i = tid; i < cnt; i += kThreads) {
        int kb = bl[i];
        if (kb >= 0 && kb <= qb0 + half) atomicOr(&dst[kb >> 5], 1u << (kb & 31));
      }
    }
  }
  __syncthreads();
  if (pattern != RS_BLOCK_SPARSE) {
    for (int wd = tid; wd < nb_words; wd += kThreads) {
      uint32_t lo = 0, hi = 0;
      if (pattern == RS_DENSE) {
        lo = range_mask(0, qb0, wd);
        hi = range_mask(0, qb0 + 1, wd);
      } else if (pattern == RS_A_SHAPE) {
        const int n_sink = cand.b0, win = cand.b1;
        const uint32_t sink0 = (n_sink > 0) ? range_mask(0, min(qb0, (n_sink - 1) >> 6), wd) : 0u;
        const uint32_t sink1 = (n_sink > 0) ? range_mask(0, min(qb0 + 1, (n_sink - 1) >> 6), wd) : 0u;
        lo = sink0 | range_mask(max(0, i0 - win + 1) >> 6, qb0, wd);
        hi = sink1 | range_mask(max(0, i0 + 64 - win + 1) >> 6, qb0 + 1, wd);
      } else {   // vertical-slash: block kb is wanted by query block qb when (qb - kb) is in D
        // bit b of the word stands for kb = 32 wd + b, i.e. for the diagonal qb - 32 wd - b: the word is a 32-bit
        // window of D, read backwards
        auto d_window = [&](int pos) -> uint32_t {      // D[pos .. pos + 31]; diagonals outside [0, 4096) are not in D
          const int w0 = pos >> 5;                      // arithmetic shift: floor
          const uint32_t a = (w0 >= 0 && w0 < 128) ? d_bits[w0] : 0u;
          const uint32_t b = (w0 + 1 >= 0 && w0 + 1 < 128) ? d_bits[w0 + 1] : 0u;
          return __funnelshift_r(a, b, (uint32_t)(pos & 31));
        };
        lo = __brev(d_window(qb0 - 32 * wd - 31));
        hi = __brev(d_window(qb0 + 1 - 32 * wd - 31));
      }
      lo_bits[wd] = lo;
      hi_bits[wd] = has_hi ? hi : 0u;
    }
  }
  __syncthreads();
  if (warp == 0) {
    // exclusive prefix of the words' chunk counts: a warp scan, 32 words at a time
    int carry = 0;
    for (int wbase = 0; wbase < nb_words; wbase += 32) {
      const int wd = wbase + lane;
      const int c = wd < nb_words ? __popc(lo_bits[wd] | hi_bits[wd]) : 0;
      int incl = c;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
      }
      if (wd < nb_words) wprefix[wd] = carry + incl - c;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) misc[2] = carry;
  } else if (pattern == RS_VERTICAL_SLASH && n_vcols > 0) {
    // The other five warps walk the ascending list of gathered columns, 32 at a time.  Columns with j <= last valid
    // row are a prefix: they are counted.  Per 32-column piece and row half: which columns survive for every row of
    // the half (valid entry, key block not after the half's block, not already covered by a block diagonal of D) and
    // which of them lie in the half's own key block; a chunk whose 64 columns all survive outside the own block needs
    // no mask at all.
    const int* vc = P.idx.vs_cols + (size_t)vs_slot * P.idx.kv_cap;
    const int i_last = i0 + rows_valid - 1;
    const int n_piece = (n_vcols + 31) >> 5;
    int cnt = 0;
    for (int piece = warp - 1; piece < n_piece; piece += kThreads / 32 - 1) {
      const int vi = piece * 32 + lane;
      const bool valid = vi < n_vcols;
      const int j = valid ? vc[vi] : 0;
      cnt += (valid && j <= i_last) ? 1 : 0;
      if (piece < 2 * kMaskChunks) {
        uint32_t kp[2], dg[2];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int dlt = qb0 + hf - (j >> 6);
          const bool covered = dlt >= 0 && dlt < 4096 && ((d_bits[dlt >> 5] >> (dlt & 31)) & 1u);
          const bool keep = valid && dlt >= 0 && !covered;
          kp[hf] = __ballot_sync(0xffffffffu, keep);
          dg[hf] = __ballot_sync(0xffffffffu, keep && dlt == 0);
        }
        if (lane == 0) {
          uint32_t* k32 = reinterpret_cast<uint32_t*>(vkeep);
          uint32_t* d32 = reinterpret_cast<uint32_t*>(vdiag);
          const int chunk = piece >> 1, part = piece & 1;
          k32[(chunk * 2 + 0) * 2 + part] = kp[0]; k32[(chunk * 2 + 1) * 2 + part] = kp[1];
          d32[(chunk * 2 + 0) * 2 + part] = dg[0]; d32[(chunk * 2 + 1) * 2 + part] = dg[1];
        }
      }
    }
    // an odd number of pieces: the second half of the last chunk holds no column
    if (warp == 1 && lane == 0 && (n_piece & 1) && n_piece < 2 * kMaskChunks) {
      uint32_t* k32 = reinterpret_cast<uint32_t*>(vkeep);
      uint32_t* d32 = reinterpret_cast<uint32_t*>(vdiag);
      const int chunk = n_piece >> 1;
      k32[(chunk * 2 + 0) * 2 + 1] = 0u; k32[(chunk * 2 + 1) * 2 + 1] = 0u;
      d32[(chunk * 2 + 0) * 2 + 1] = 0u; d32[(chunk * 2 + 1) * 2 + 1] = 0u;
    }
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (lane == 0 && cnt > 0) atomicAdd(const_cast<int*>(&misc[3]), cnt);
  }
  __syncthreads();
  for (int wd = tid; wd < nb_words; wd += kThreads) {
    uint32_t lo = lo_bits[wd], hi = hi_bits[wd], any = lo | hi;
    int at = wprefix[wd];
    while (any) {
      const int b = __ffs(any) - 1;
      any &= any - 1;
      const int kb = 32 * wd + b;
      uint32_t e = (uint32_t)kb;
      if ((lo >> b) & 1u) e |= F_LO;
      if ((hi >> b) & 1u) e |= F_HI;
      if (kb >= qb0) e |= F_CAUSAL;
      if (pattern == RS_A_SHAPE) {
        const bool in_window = kb * 64 >= i0 + kTileM - cand.b1;
        const bool in_sink = (kb + 1) * 64 <= cand.b0;
        if (!in_window && !in_sink) e |= F_EDGE;
      }
      list[at++] = (uint16_t)e;
    }
  }
  __syncthreads();
  const int n_block = misc[2], n_vert = (misc[3] + kChunk - 1) / kChunk;     // misc[3]: visible gathered columns
  const int n_chunks = n_block + n_vert;
  // =========================================================================================== roles
  // Everything below is pipelined per 64-key chunk; chunk c uses slot c & 1 of the K / V rings, of the two 64-column
  // score buffers in TMEM and of the barrier pairs, in phase (c >> 1) & 1.  While the softmax warps work on chunk c the
  // tensor pipe runs O += P(c-1) V(c-1) and S(c+1) = Q K(c+1)^T, so neither side waits for the other in steady state.
  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      bool ok = true;
      int site = 1;
      auto load_chunk = [&](int ch, uint32_t dst, uint32_t bar, const CUtensorMap* tm_blocks, const CUtensorMap* tm_packed) {
        mbar_arrive_expect_tx(bar, 16384u);
        if (ch < n_block) {
          const int row = g * P.n + (int)(list[ch] & 0xfffu) * kChunk;
          tma_load_2d(dst, tm_blocks, bar, 0, row);
          tma_load_2d(dst + 16384, tm_blocks, bar, 64, row);
        } else {
          const int row = item * P.kv_pad + (ch - n_block) * kChunk;
          tma_load_2d(dst, tm_packed, bar, 0, row);
          tma_load_2d(dst + 16384, tm_packed, bar, 64, row);
        }
      };
      // order of the loads = order in which their slots come free: K0 K1 V0 K2 V1 K3 ...
      for (int i = 0; i < n_chunks + 2 && ok; ++i) {
        if (i >= 2) {
          const int ch = i - 2;
          const uint32_t slot = (uint32_t)(ch & 1), ph = (uint32_t)((ch >> 1) & 1);
          ok = mbar_wait(bar_ve + 8u * slot, ph ^ 1u, abort_flag); site = 2;
          if (!ok) break;
          load_chunk(ch, base + SmemLayout::v + slot * 8192u, bar_vf + 8u * slot, &tmV, &tmVp);
        }
        if (i < n_chunks) {
          const uint32_t slot = (uint32_t)(i & 1), ph = (uint32_t)((i >> 1) & 1);
          ok = mbar_wait(bar_ke + 8u * slot, ph ^ 1u, abort_flag); site = 1;
          if (!ok) break;
          load_chunk(i, base + SmemLayout::k + slot * 8192u, bar_kf + 8u * slot, &tmK, &tmKp);
        }
      }
      if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, site); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      const uint32_t d_s = tmem + kColS, d_o = tmem + kColO;
      // Descriptor words are formed once; an instruction then costs the issuing thread two adds and the MMA itself.
      const uint64_t q_desc = umma_smem_desc(base + SmemLayout::q, 16, 1024);
      const uint64_t k_desc = umma_smem_desc(base + SmemLayout::k, 16, 1024);
      const uint64_t v_desc = umma_smem_desc(base + SmemLayout::v, 16384, 1024);
      const uint32_t q_lo = (uint32_t)q_desc, q_hi = (uint32_t)(q_desc >> 32);
      const uint32_t k_lo = (uint32_t)k_desc, k_hi = (uint32_t)(k_desc >> 32);
      const uint32_t v_lo = (uint32_t)v_desc, v_hi = (uint32_t)(v_desc >> 32);
      constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 64, 0, 0);
      constexpr uint32_t kIdescPV = umma_idesc_bf16(128, 128, 0, 1);
      auto issue_qk = [&](uint32_t slot) {      // S[slot] = Q K[slot]^T: 8 steps of 16 head dimensions
        const uint32_t kb = k_lo + slot * 512u, ds = d_s + slot * 64u;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (uint32_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
          umma_ss2(ds, q_lo + off, q_hi, kb + off, k_hi, kIdescQK, kk > 0 ? 1u : 0u);
        }
      };
      auto issue_pv = [&](uint32_t slot, bool accumulate) {   // O += P[slot] V[slot]: 4 steps of 16 keys
        const uint32_t vb = v_lo + slot * 512u, ps = d_s + slot * 64u;
        umma_ts2(d_o, ps, vb, v_hi, kIdescPV, accumulate ? 1u : 0u);
#pragma unroll
        for (int kk = 1; kk < 4; ++kk) umma_ts2(d_o, ps + 8u * kk, vb + 128u * kk, v_hi, kIdescPV, 1u);
      };
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      int site = 3;
      for (int c = 0; c < 2 && c < n_chunks && ok; ++c) {
        ok = mbar_wait(bar_kf + 8u * c, 0, abort_flag); site = 4;
        if (!ok) break;
        tc_fence_after();
        issue_qk((uint32_t)c);
        umma_commit(bar_s + 8u * c);
        umma_commit(bar_ke + 8u * c);
      }
      for (int c = 0; c < n_chunks && ok; ++c) {
        const uint32_t slot = (uint32_t)(c & 1), ph = (uint32_t)((c >> 1) & 1);
        ok = mbar_wait(bar_p + 8u * slot, ph, abort_flag); site = 5;
        if (!ok) break;
        ok = mbar_wait(bar_vf + 8u * slot, ph, abort_flag); site = 6;
        if (!ok) break;
        tc_fence_after();
        issue_pv(slot, c > 0);
        umma_commit(bar_ve + 8u * slot);
        if (c + 2 < n_chunks) {
          ok = mbar_wait(bar_kf + 8u * slot, ph ^ 1u, abort_flag); site = 7;
          if (!ok) break;
          tc_fence_after();
          issue_qk(slot);
          umma_commit(bar_s + 8u * slot);
          umma_commit(bar_ke + 8u * slot);
        }
      }
      if (ok) umma_commit(bar_o);
      if (!ok) { rs_report(P.status, RS_ERR_TIMEOUT, site); *abort_flag = 1; }
    }
  } else {
    // -------------------------------------------------------------------- softmax / correction / epilogue
    const int quad = warp & 3;
    const int r = quad * 32 + lane;            // row of the tile = TMEM lane
    const int i = i0 + r;                      // global query row
    const int half = r >> 6;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t t_s = tmem + lane_addr + kColS, t_o = tmem + lane_addr + kColO;
    const float sl2 = P.scale_log2e;
    const float NEG_INF = -INFINITY;
    float m_run = NEG_INF, l_run = 0.f;
    const int* vcols = P.idx.vs_cols + (size_t)vs_slot * P.idx.kv_cap;
    bool ok = true;
    uint32_t v[32], v2[32];
    auto max3 = [](float a, float b, float c) -> float {
      float d;
      asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
      return d;
    };
    auto max32 = [&](const uint32_t (&x)[32]) -> float {
      float mx0 = max3(__uint_as_float(x[0]), __uint_as_float(x[1]), __uint_as_float(x[2]));
      float mx1 = max3(__uint_as_float(x[3]), __uint_as_float(x[4]), __uint_as_float(x[5]));
      float mx2 = max3(__uint_as_float(x[6]), __uint_as_float(x[7]), __uint_as_float(x[8]));
      float mx3 = max3(__uint_as_float(x[9]), __uint_as_float(x[10]), __uint_as_float(x[11]));
#pragma unroll
      for (int q = 12; q < 28; q += 8) {
        mx0 = max3(mx0, __uint_as_float(x[q]), __uint_as_float(x[q + 1]));
        mx1 = max3(mx1, __uint_as_float(x[q + 2]), __uint_as_float(x[q + 3]));
        mx2 = max3(mx2, __uint_as_float(x[q + 4]), __uint_as_float(x[q + 5]));
        mx3 = max3(mx3, __uint_as_float(x[q + 6]), __uint_as_float(x[q + 7]));
      }
      mx0 = max3(mx0, __uint_as_float(x[28]), __uint_as_float(x[29]));
      mx1 = max3(mx1, __uint_as_float(x[30]), __uint_as_float(x[31]));
      return fmaxf(max3(mx0, mx1, mx2), mx3);
    };
    auto exp_chunk = [&](const uint32_t (&x)[32], uint32_t dst, float m_use) {
      uint32_t pk[16];
      uint64_t acc = 0ull, acc_b = 0ull;     // two packed pairs of fp32 partial sums
      uint64_t sl2x2, negm2;
      asm("mov.b64 %0, {%1, %1};" : "=l"(sl2x2) : "f"(sl2));
      asm("mov.b64 %0, {%1, %1};" : "=l"(negm2) : "f"(-m_use));
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        uint64_t s2, t2, p2;
        asm("mov.b64 %0, {%1, %2};" : "=l"(s2) : "r"(x[2 * q]), "r"(x[2 * q + 1]));
        asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t2) : "l"(s2), "l"(sl2x2), "l"(negm2));
        float t0, t1;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(t0), "=f"(t1) : "l"(t2));
        const float p0 = fast_exp2(t0), p1 = fast_exp2(t1);
        asm("mov.b64 %0, {%1, %2};" : "=l"(p2) : "f"(p0), "f"(p1));
        if (q & 1) { asm("add.rn.f32x2 %0, %1, %2;" : "=l"(acc_b) : "l"(acc_b), "l"(p2)); }
        else       { asm("add.rn.f32x2 %0, %1, %2;" : "=l"(acc) : "l"(acc), "l"(p2)); }
        pk[q] = pack_bf16x2(p0, p1);
      }
      asm("add.rn.f32x2 %0, %1, %2;" : "=l"(acc) : "l"(acc), "l"(acc_b));
      float a0, a1;
      asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc));
      l_run += a0 + a1;
      tmem_st16(dst, pk);
    };

    // One pass per 64-key chunk: rare chunks are masked in place first, then the scores go to registers (two
    // 32-column loads per wait), chunk maximum, P = exp2(S * scale*log2e - m) against the running maximum, bf16 P
    // over the start of the chunk's score buffer.  The maximum only moves when some row of the warp exceeds it by more
    // than 2^8; then l and O are rescaled, after the product of the previous chunk has left the tensor pipe.
    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t slot = (uint32_t)(ch & 1), ph = (uint32_t)((ch >> 1) & 1);
      const uint32_t t_sc = t_s + slot * 64u;
      ok = mbar_wait(bar_s + 8u * slot, ph, abort_flag);
      if (!ok) break;
      tc_fence_after();
      {
        int mode = -1, j0 = 0, edge = 0, vbase = 0;
        unsigned long long vk = 0ull, vd = 0ull;
        if (ch < n_block) {
          const uint32_t e = list[ch];
          if (!(e & (half ? F_HI : F_LO))) {
            mode = 0;
          } else if (e & (F_CAUSAL | F_EDGE)) {
            mode = 1;
            j0 = (int)(e & 0xfffu) * kChunk;
            edge = (e & F_EDGE) ? 1 : 0;
          }
        } else {
          const int vch = ch - n_block;
          vbase = vch * kChunk;
          if (vch < kMaskChunks) {
            vk = vkeep[vch * 2 + half];
            vd = vdiag[vch * 2 + half];
            mode = (vk == ~0ull && vd == 0ull) ? -1 : 3;
          } else {
            mode = 2;
          }
        }
        if (mode == 0) {
          // this half of the tile does not take the chunk (uniform over the warp): its probabilities are zeros and
          // neither the running maximum nor the sum moves, so nothing is loaded or exponentiated
          uint32_t z[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) z[q] = 0u;
          tmem_st16(t_sc, z);
          tmem_st16(t_sc + 16u, z);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(bar_p + 8u * slot);
          continue;
        }
        if (mode >= 0) rs_mask_chunk(t_sc, mode, i, j0, edge, cand.b0, cand.b1, vcols, vbase, n_vcols, d_bits, vk, vd);
      }
      tmem_ld32(t_sc, v);
      tmem_ld32(t_sc + 32u, v2);
      tc_wait_ld();
      const float m_chunk = fmaxf(max32(v), max32(v2)) * sl2;
      const float m_new = fmaxf(m_run, m_chunk);
      const bool need = m_new > m_run + 8.0f;
      if (__any_sync(0xffffffffu, need)) {
        const float alpha = (m_new == NEG_INF) ? 1.0f : fast_exp2(m_run - m_new);
        l_run *= alpha;
        m_run = m_new;
        if (ch > 0) {
          // O holds the products up to chunk ch - 1; the last of them may still be in flight
          const uint32_t pslot = (uint32_t)((ch - 1) & 1), pph = (uint32_t)(((ch - 1) >> 1) & 1);
          ok = mbar_wait(bar_ve + 8u * pslot, pph, abort_flag);
          if (!ok) break;
          tc_fence_after();
          uint32_t w32[32];
#pragma unroll 1
          for (int c4 = 0; c4 < 4; ++c4) {
            tmem_ld32(t_o + (uint32_t)c4 * 32u, w32);
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < 32; ++q) w32[q] = __float_as_uint(__uint_as_float(w32[q]) * alpha);
            tmem_st32(t_o + (uint32_t)c4 * 32u, w32);
          }
          tc_wait_st();
        }
      }
      const float m_use = (m_run == NEG_INF) ? 0.f : m_run;
      exp_chunk(v, t_sc, m_use);
      exp_chunk(v2, t_sc + 16u, m_use);
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p + 8u * slot);
    }

    if (ok) ok = mbar_wait(bar_o, 0, abort_flag);
    if (ok) {
      tc_fence_after();
      const float inv = (l_run > 0.f) ? 1.0f / l_run : 0.f;
      const bool valid = r < rows_valid;
      float ss = 0.f;
      const size_t orow = ((size_t)h * P.n + (size_t)i) * RS_HEAD_DIM;
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        tmem_ld32(t_o + (uint32_t)c4 * 32u, v);
        tc_wait_ld();
        float f[32];
#pragma unroll
        for (int x = 0; x < 32; ++x) { f[x] = __uint_as_float(v[x]) * inv; ss = fmaf(f[x], f[x], ss); }
        if (valid) {
          if (P.o_f32) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(P.O) + orow + c4 * 32);
#pragma unroll
            for (int x = 0; x < 8; ++x) dst[x] = make_float4(f[4 * x], f[4 * x + 1], f[4 * x + 2], f[4 * x + 3]);
          } else {
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(P.O) + orow + c4 * 32);
#pragma unroll
            for (int x = 0; x < 4; ++x)
              dst[x] = make_uint4(pack_bf16x2(f[8 * x], f[8 * x + 1]), pack_bf16x2(f[8 * x + 2], f[8 * x + 3]),
                                  pack_bf16x2(f[8 * x + 4], f[8 * x + 5]), pack_bf16x2(f[8 * x + 6], f[8 * x + 7]));
          }
        }
      }
      if (valid) {
        const size_t ridx = (size_t)h * P.n + (size_t)i;
        P.lse[ridx] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        if (P.onorm != nullptr) P.onorm[ridx] = sqrtf(ss);
      }
    } else if (lane == 0 && quad == 0) {
      rs_report(P.status, RS_ERR_TIMEOUT, 8);
      *abort_flag = 1;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && P.counters != nullptr) {
    atomicAdd(&P.counters[0], (unsigned long long)n_chunks);
    atomicAdd(&P.counters[1], 1ull);
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// -------------------------------------------------------------------------------------------- work list
// Estimated number of 64-key chunks of work item wid = (head, tile of the head), used only to order the launch.
__device__ __forceinline__ int rs_tile_cost(const AttnParams& P, int wid, int2* item_tile) {
  const int h = wid / P.tiles_per_head;
  const int tt = wid - h * P.tiles_per_head;
  int s = 0;
  while (s + 1 < P.n_seg && tt >= P.tile_base[s + 1]) ++s;
  const int tile = tt - P.tile_base[s];
  const int item = s * P.Hq + h;
  const int q0 = P.seg_bounds[s], q1 = P.seg_bounds[s + 1];
  const int i0 = q0 + tile * kTileM;
  const int rows_valid = min(kTileM, q1 - i0);
  const int qb0 = i0 >> 6;
  const int qb_last = rows_valid > kChunk ? qb0 + 1 : qb0;
  const rs_candidate cand = (P.choice != nullptr) ? P.lib[P.choice[item]] : rs_candidate{RS_DENSE, 0, 0, 0};
  int c = qb_last + 1;
  if (cand.pattern == RS_A_SHAPE) {
    c = min(qb_last + 1, (cand.b0 + 63) / 64 + (cand.b1 + 63) / 64 + 2);
  } else if (cand.pattern == RS_VERTICAL_SLASH) {
    const int slot = P.vs_eval_layout ? item * P.n_cand + P.choice[item] : item;
    const int* cnt = P.idx.vs_count + 4 * slot;
    const int* dl = P.idx.vs_diag + (size_t)slot * P.idx.nd_cap;
    int lo = 0, hi = cnt[2];
    while (lo < hi) { int mid = (lo + hi) >> 1; if (dl[mid] <= qb_last) lo = mid + 1; else hi = mid; }
    c = min(qb_last + 1, lo + 1) + (cnt[0] + 63) / 64;
  } else if (cand.pattern == RS_BLOCK_SPARSE) {
    const size_t row = (size_t)h * (P.n >> 6) + qb0;
    c = P.idx.bs_count[row] + (qb_last > qb0 ? P.idx.bs_count[row + 1] : 0);
  }
  *item_tile = make_int2(item, tile);
  return c;
}

// Preparation of the launch, one kernel with two kinds of blocks.
// Blocks 0 .. n_groups-1: the work list (Section 3.4: heads are grouped into one launch).  When K and V of all heads
// exceed L2, n_groups = Hkv: KV groups run one after the other (the CTAs in flight then stream the same K / V, which
// keeps them in L2), inside a group the heaviest item first.  When they fit, n_groups = 1: heaviest item first over the
// whole launch (no long tile of the last group is left to start late).  One block per group: cost of each of the
// group's items (they are contiguous in the head-major enumeration), then a counting sort by cost.  cost / items are
// scratch of the block itself.
// Blocks n_groups ..: the vertical key / value rows of every vertical-slash item are gathered into a contiguous,
// zero-padded buffer; pack_blocks blocks per item, 64 rows each (16 threads move one 256-byte row).
__global__ void __launch_bounds__(1024)
rs_attn_prepare_kernel(AttnParams P, int n_groups, int per_group, int n_bins, int* cost, int2* items, int2* order,
                       int pack_blocks, const __nv_bfloat16* K, const __nv_bfloat16* V, __nv_bfloat16* Kp,
                       __nv_bfloat16* Vp) {
  extern __shared__ int hist[];
  if ((int)blockIdx.x >= n_groups) {
    const int pb = blockIdx.x - n_groups;
    const int item = pb / pack_blocks;
    if (P.choice == nullptr || P.lib[P.choice[item]].pattern != RS_VERTICAL_SLASH) return;
    const int h = item % P.Hq, g = h / P.group;
    const int slot = P.vs_eval_layout ? item * P.n_cand + P.choice[item] : item;
    const int n_cols = P.idx.vs_count[4 * slot];
    const int row = (pb - item * pack_blocks) * 64 + (threadIdx.x >> 4);
    if (row >= P.kv_pad) return;
    const int l16 = threadIdx.x & 15;
    uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
    if (row < n_cols) {
      const int j = P.idx.vs_cols[(size_t)slot * P.idx.kv_cap + row];
      const size_t src = ((size_t)g * P.n + (size_t)j) * RS_HEAD_DIM;
      kv = reinterpret_cast<const uint4*>(K + src)[l16];
      vv = reinterpret_cast<const uint4*>(V + src)[l16];
    }
    const size_t dst = ((size_t)item * P.kv_pad + row) * RS_HEAD_DIM;
    reinterpret_cast<uint4*>(Kp + dst)[l16] = kv;
    reinterpret_cast<uint4*>(Vp + dst)[l16] = vv;
    return;
  }
  const int base = blockIdx.x * per_group;
  cost += base; items += base; order += base;
  for (int i = threadIdx.x; i <= n_bins; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < per_group; i += blockDim.x) {
    int2 it;
    const int c = min(rs_tile_cost(P, base + i, &it), n_bins - 1);
    cost[i] = c;
    items[i] = it;
    atomicAdd(&hist[c], 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int b = n_bins - 1; b >= 0; --b) { int c = hist[b]; hist[b] = acc; acc += c; }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < per_group; i += blockDim.x) {
    const int pos = atomicAdd(&hist[cost[i]], 1);
    order[pos] = items[i];
  }
}

size_t attn_smem_bytes(int n) {
  const int list_cap = (n >> 6) + 64;
  return 1024 + SmemLayout::end_tiles + ((list_cap * 2 + 15) & ~15) + 3 * 128 * 4 + 132 * 4 + 14 * 8 + 64 + 4 * kMaskChunks * 8;
}

struct WsPlan { size_t cost, items, order, kpack, vpack, total; int n_work, kv_pad, n_items; };

WsPlan plan_ws(const rs_problem* p, int max_kv) {
  WsPlan w{};
  int tiles = 0;
  for (int s = 0; s < p->n_segments; ++s) tiles += (p->seg_bounds[s + 1] - p->seg_bounds[s] + kTileM - 1) / kTileM;
  w.n_work = tiles * p->n_q_heads;
  w.n_items = p->n_segments * p->n_q_heads;
  w.kv_pad = (int)rs_align_up((size_t)(max_kv > 0 ? max_kv : 0), 64);
  size_t off = 0;
  w.cost = off;  off += rs_align_up((size_t)w.n_work * 4, 256);
  w.items = off; off += rs_align_up((size_t)w.n_work * 8, 256);
  w.order = off; off += rs_align_up((size_t)w.n_work * 8, 256);
  const size_t pack = rs_align_up((size_t)w.n_items * (size_t)(w.kv_pad > 0 ? w.kv_pad : 64) * RS_HEAD_DIM * 2, 256);
  w.kpack = off; off += pack;
  w.vpack = off; off += pack;
  w.total = off;
  return w;
}

constexpr size_t kL2ResidentBytes = 96ull << 20;     // K + V of all heads below this: they stay in the 126 MB L2

// Scratch of one attention launch: the work list (cost, items, launch order: one entry per 128-row tile) and, for
// vertical-slash items, the packed K / V rows of the gathered columns.
struct AttnScratch { int* cost; int2* items; int2* order; __nv_bfloat16 *Kp, *Vp; int kv_pad; int n_work, n_items; };

// Enqueues the preparation kernel (work list, gather of the vertical columns) and the attention launch.  Arguments are checked
// by the callers; `sc` says where the scratch lives (caller workspace or the library's built-in array).
int enqueue_attn(const rs_problem* p, const void* Q, const void* K, const void* V, const rs_candidate* lib, int n_cand,
                 const rs_index_set* idx, const int32_t* choice, bool any_vs, bool vs_eval_layout, void* O, int o_dtype,
                 float* lse, float* onorm, uint64_t* counters, const AttnScratch& sc, int32_t* status,
                 cudaStream_t stream) {
  AttnParams P{};
  P.n = p->n_keys; P.Hq = p->n_q_heads; P.Hkv = p->n_kv_heads; P.group = p->n_q_heads / p->n_kv_heads;
  P.n_seg = p->n_segments; P.n_cand = n_cand;
  int tiles = 0;
  for (int s = 0; s <= p->n_segments; ++s) {
    P.seg_bounds[s] = p->seg_bounds[s];
    P.tile_base[s] = tiles;
    if (s < p->n_segments) tiles += (p->seg_bounds[s + 1] - p->seg_bounds[s] + kTileM - 1) / kTileM;
  }
  P.tiles_per_head = tiles;
  for (int c = 0; c < n_cand; ++c) P.lib[c] = lib[c];
  P.choice = choice;
  if (idx) P.idx = *idx;
  P.vs_eval_layout = vs_eval_layout ? 1 : 0;
  P.kv_pad = sc.kv_pad;
  P.order = sc.order;
  P.O = O; P.o_f32 = o_dtype; P.lse = lse; P.onorm = onorm;
  P.counters = reinterpret_cast<unsigned long long*>(counters);
  P.status = status;
  P.scale_log2e = (float)(1.4426950408889634 / sqrt((double)RS_HEAD_DIM));

  CUtensorMap tmQ, tmK, tmV, tmKp, tmVp;
  if (rs_make_tmap_bf16_2d(&tmQ, Q, (uint64_t)P.Hq * P.n, RS_HEAD_DIM, kTileM, 64) ||
      rs_make_tmap_bf16_2d(&tmK, K, (uint64_t)P.Hkv * P.n, RS_HEAD_DIM, kChunk, 64) ||
      rs_make_tmap_bf16_2d(&tmV, V, (uint64_t)P.Hkv * P.n, RS_HEAD_DIM, kChunk, 64))
    return RS_ERR_CUDA;
  if (sc.Kp != nullptr) {
    const uint64_t pack_rows = (uint64_t)sc.n_items * (uint64_t)sc.kv_pad;
    if (rs_make_tmap_bf16_2d(&tmKp, sc.Kp, pack_rows, RS_HEAD_DIM, kChunk, 64) ||
        rs_make_tmap_bf16_2d(&tmVp, sc.Vp, pack_rows, RS_HEAD_DIM, kChunk, 64))
      return RS_ERR_CUDA;
  } else {          // no gathered columns in this launch: the packed maps are never read and alias K and V
    tmKp = tmK; tmVp = tmV;
  }

  const int n_work = sc.n_work;
  // every entry of cost / items / order is rewritten by the kernel below, so nothing has to be cleared
  const int n_bins = (P.n >> 6) + 66;
  const bool pack = choice != nullptr && any_vs && sc.Kp != nullptr;
  const int pack_blocks = pack ? (P.kv_pad + 63) / 64 : 0;
  const size_t kv_bytes = 2ull * (size_t)P.Hkv * (size_t)P.n * RS_HEAD_DIM * sizeof(__nv_bfloat16);
  const int n_groups = (kv_bytes <= kL2ResidentBytes || n_work % P.Hkv != 0) ? 1 : P.Hkv;
  rs_attn_prepare_kernel<<<n_groups + pack_blocks * sc.n_items, 1024, (n_bins + 1) * sizeof(int), stream>>>(
      P, n_groups, n_work / n_groups, n_bins, sc.cost, sc.items, sc.order, pack_blocks,
      reinterpret_cast<const __nv_bfloat16*>(K), reinterpret_cast<const __nv_bfloat16*>(V), sc.Kp, sc.Vp);
  if (rs_ensure_dynamic_smem(g_attn_smem, rs_attn_kernel, 116 * 1024) != RS_OK) return RS_ERR_CUDA;
  rs_attn_kernel<<<n_work, kThreads, attn_smem_bytes(P.n), stream>>>(tmQ, tmK, tmV, tmKp, tmVp, P);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}

int launch_attn(const rs_problem* p, const void* Q, const void* K, const void* V, const rs_candidate* lib,
                int n_cand, const rs_index_set* idx, const int32_t* choice, void* O, int o_dtype, float* lse,
                float* onorm, uint64_t* counters, void* ws, size_t ws_bytes, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !K || !V || !O || !lse || !ws) return RS_ERR_INVALID_ARG;
  if (n_cand < 0 || n_cand > RS_MAX_CANDIDATES) return RS_ERR_INVALID_ARG;
  if (choice != nullptr && (lib == nullptr || idx == nullptr || n_cand == 0)) return RS_ERR_INVALID_ARG;
  rc = rs_check_device();
  if (rc != RS_OK) return rc;

  int max_kv = 0;
  bool any_vs = false;
  for (int c = 0; c < n_cand; ++c) {
    if (lib[c].pattern == RS_VERTICAL_SLASH) { any_vs = true; if (lib[c].b0 > max_kv) max_kv = lib[c].b0; }
    if (lib[c].pattern == RS_A_SHAPE && (lib[c].b1 < 1 || lib[c].b0 < 0)) return RS_ERR_INVALID_ARG;
    if (lib[c].pattern < 0 || lib[c].pattern > 3) return RS_ERR_INVALID_ARG;
  }
  if (max_kv > p->n_keys) max_kv = p->n_keys;      // a column list never holds more than n_keys entries
  bool vs_eval_layout = false;
  if (choice != nullptr && any_vs) {
    const int n_items_ = p->n_segments * p->n_q_heads;
    if (idx->kv_cap < max_kv || idx->n_vs_slots < n_items_) return RS_ERR_INVALID_ARG;
    vs_eval_layout = n_cand > 1 && idx->n_vs_slots == n_items_ * n_cand;
  }
  const WsPlan w = plan_ws(p, max_kv);
  if (ws_bytes < w.total) return RS_ERR_WORKSPACE_TOO_SMALL;
  if (((uintptr_t)ws & 255) != 0) return RS_ERR_INVALID_ARG;
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);
  AttnScratch sc{reinterpret_cast<int*>(wsb + w.cost), reinterpret_cast<int2*>(wsb + w.items),
                 reinterpret_cast<int2*>(wsb + w.order), reinterpret_cast<__nv_bfloat16*>(wsb + w.kpack),
                 reinterpret_cast<__nv_bfloat16*>(wsb + w.vpack), w.kv_pad > 0 ? w.kv_pad : 64, w.n_work, w.n_items};
  return enqueue_attn(p, Q, K, V, lib, n_cand, idx, choice, any_vs, vs_eval_layout, O, o_dtype, lse, onorm, counters, sc,
                      status, (cudaStream_t)stream_);
}

}  // namespace

size_t rs_attn_workspace_bytes(const rs_problem* p, int max_kv) { return plan_ws(p, max_kv).total; }

extern "C" int rs_sparse_prefill_attn(const rs_problem* p, const void* Q, const void* K, const void* V,
                                      const rs_candidate* lib, int n_cand, const rs_index_set* idx,
                                      const int32_t* choice, void* O, int o_dtype, float* lse_sel, float* onorm,
                                      uint64_t* counters, void* ws, size_t ws_bytes, int32_t* status, void* stream) {
  if (!lib || !idx || !choice || n_cand <= 0) return RS_ERR_INVALID_ARG;
  return launch_attn(p, Q, K, V, lib, n_cand, idx, choice, O, o_dtype, lse_sel, onorm, counters, ws, ws_bytes, status,
                     stream);
}

extern "C" int rs_dense_prefill_attn(const rs_problem* p, const void* Q, const void* K, const void* V, void* O,
                                     int o_dtype, float* lse, float* onorm, uint64_t* counters, void* ws,
                                     size_t ws_bytes, int32_t* status, void* stream) {
  return launch_attn(p, Q, K, V, nullptr, 0, nullptr, nullptr, O, o_dtype, lse, onorm, counters, ws, ws_bytes, status,
                     stream);
}

// ---------------------------------------------------------------------------------------------------------------
// Dense causal attention without a caller workspace.
//
// Some callers cannot hand the library a scratch buffer because they cannot allocate device memory at the point of
// the call: code running inside a framework's memory-pool callback, a plugin that is given only its input and
// output tensors, or a latency-critical serving loop in which any cudaMalloc (which synchronises the device) is
// forbidden.  For them the work list of the attention launch lives in a fixed array inside this library image.
// The array is part of the module, so every GPU that loads the library holds these bytes until the process exits.
namespace {

constexpr int kNoAllocMaxTiles = 16384;                         // (query heads) x (128-row query tiles) per call
constexpr size_t kNoAllocBytes = (size_t)kNoAllocMaxTiles * 20; // cost (4 B) + items (8 B) + order (8 B) per tile
static __device__ __align__(256) unsigned char rs_noalloc_scratch[kNoAllocBytes];

// In host code the array's name is only a handle for the runtime; the device address must be asked for, once per
// device and with that device current.
int noalloc_scratch_ptr(void** out) {
  static void* cached[64] = {nullptr};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RS_ERR_CUDA;
  if (dev < 0 || dev >= 64) return RS_ERR_UNSUPPORTED_DEVICE;
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, rs_noalloc_scratch) != cudaSuccess || ptr == nullptr) return RS_ERR_CUDA;
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return RS_OK;
}

}  // namespace

extern "C" int rs_dense_prefill_attn_noalloc(const rs_problem* p, const void* Q, const void* K, const void* V, void* O,
                                             int o_dtype, float* lse, float* onorm, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !K || !V || !O || !lse) return RS_ERR_INVALID_ARG;
  int tiles = 0;
  for (int s = 0; s < p->n_segments; ++s) tiles += (p->seg_bounds[s + 1] - p->seg_bounds[s] + kTileM - 1) / kTileM;
  const long long n_work_ll = (long long)tiles * p->n_q_heads;
  if (n_work_ll > kNoAllocMaxTiles) return RS_ERR_NOALLOC_TOO_LARGE;
  rc = rs_check_device();
  if (rc != RS_OK) return rc;
  void* scratch = nullptr;
  rc = noalloc_scratch_ptr(&scratch);
  if (rc != RS_OK) return rc;
  unsigned char* sb = reinterpret_cast<unsigned char*>(scratch);
  AttnScratch sc{reinterpret_cast<int*>(sb), reinterpret_cast<int2*>(sb + (size_t)kNoAllocMaxTiles * 4),
                 reinterpret_cast<int2*>(sb + (size_t)kNoAllocMaxTiles * 12), nullptr, nullptr, 64, (int)n_work_ll,
                 p->n_segments * p->n_q_heads};
  // the same enqueue as rs_dense_prefill_attn: same kernels, same work list, only the scratch lives elsewhere
  return enqueue_attn(p, Q, K, V, nullptr, 0, nullptr, nullptr, false, false, O, o_dtype, lse, onorm, nullptr, sc, status,
                      (cudaStream_t)stream_);
}
