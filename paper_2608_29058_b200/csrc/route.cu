// Risk score (Eq. 4), greedy substitution for the budgeted routing problem (Eq. 6-8), fallback walk and forced
// dense (Section 3.4), solved by one thread block so that no host round trip sits between probe and attention.
//
// Exactness: coverage and cost are integers, so totals are exact; risks are IEEE doubles built from separately
// rounded operations (no fused multiply-add); a substitution's ratio is one IEEE division and candidates are
// ordered by (ratio, larger saving, lower item, lower candidate), a total order, so the parallel arg-min picks
// the same substitution as a sequential scan.
#include "common.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kMaxItems = 2048;
constexpr int kSortPairs = 2048;      // up to this many pairs the merge of the sequences is a parallel sort
constexpr int kCachePairs = 4096;     // (item, candidate) pairs whose risk / cost are kept in shared memory

struct RouteArgs {
  int n_items, n_cand, Hq, Hkv, group, dense_c;
  rs_candidate lib[RS_MAX_CANDIDATES];
  int next_larger[RS_MAX_CANDIDATES];
  const rs_cand_stats* stats;
  const int64_t* cost;
  const float* vmax;
  rs_route_params prm;
  int32_t* choice;
  rs_route_report* report;
  int32_t* status;
};

struct Sub { double ratio; long long dT; int item, k; };

__device__ __forceinline__ bool better(const Sub& a, const Sub& b) {
  if (a.k < 0) return false;
  if (b.k < 0) return true;
  if (a.ratio != b.ratio) return a.ratio < b.ratio;
  if (a.dT != b.dT) return a.dT > b.dT;
  if (a.item != b.item) return a.item < b.item;
  return a.k < b.k;
}

__device__ __forceinline__ Sub shfl_sub(const Sub& a, int off) {
  Sub r;
  r.ratio = __shfl_xor_sync(0xffffffffu, a.ratio, off);
  r.dT = __shfl_xor_sync(0xffffffffu, a.dT, off);
  r.item = __shfl_xor_sync(0xffffffffu, a.item, off);
  r.k = __shfl_xor_sync(0xffffffffu, a.k, off);
  return r;
}

__device__ __forceinline__ long long cost_of(const RouteArgs& A, int item, int c) {
  if (A.cost != nullptr) return A.cost[(size_t)item * A.n_cand + c];
  if (A.stats == nullptr) return 0;
  return (long long)(4ull * RS_HEAD_DIM * A.stats[(size_t)item * A.n_cand + c].pairs);
}

__device__ __forceinline__ double m_hat_of(const RouteArgs& A, int item, int c) {
  if (A.lib[c].pattern == RS_DENSE) return 1.0;
  const rs_cand_stats& st = A.stats[(size_t)item * A.n_cand + c];
  const unsigned long long tot = st.cov_fx[0] + st.cov_fx[1] + st.cov_fx[2] + st.cov_fx[3];
  return (double)tot / 274877906944.0;          // 64 * 2^32
}

__device__ __forceinline__ double risk_of(const RouteArgs& A, int item, int c) {
  if (A.lib[c].pattern == RS_DENSE || A.stats == nullptr) return 0.0;
  const rs_cand_stats& st = A.stats[(size_t)item * A.n_cand + c];
  double mx = 0.0, mn = 2.0;
#pragma unroll
  for (int g = 0; g < RS_PROBE_GROUPS; ++g) {
    const double mg = (double)st.cov_fx[g] / 68719476736.0;   // 16 * 2^32
    mx = fmax(mx, mg);
    mn = fmin(mn, mg);
  }
  double u = __dsub_rn(mx, mn);
  if (A.prm.cov_mix != nullptr) {
    // disagreement among the row subsets of the query mixture
    const uint64_t* cm = A.prm.cov_mix + ((size_t)item * A.n_cand + c) * 4;
    double hi = 0.0, lo = 2.0;
    bool any = false;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      if (A.prm.mix_rows[b] <= 0) continue;
      const double mb = (double)cm[b] / ((double)A.prm.mix_rows[b] * 4294967296.0);
      hi = fmax(hi, mb);
      lo = fmin(lo, mb);
      any = true;
    }
    if (any) u = __dsub_rn(hi, lo);
  }
  double r = __dadd_rn(__dsub_rn(1.0, m_hat_of(A, item, c)), __dmul_rn(A.prm.alpha, u));
  if (A.prm.e != nullptr && A.prm.beta != 0.0) r = __dadd_rn(r, __dmul_rn(A.prm.beta, A.prm.e[(size_t)item * A.n_cand + c]));
  return r;
}

__global__ void __launch_bounds__(kThreads)
rs_route_kernel(const __grid_constant__ RouteArgs A) {
  extern __shared__ unsigned char route_smem[];       // ibest[n_items] | c_risk[cache] | c_cost[cache] | ch[n_items]
  const int n_cache = (A.n_items * A.n_cand <= kCachePairs) ? A.n_items * A.n_cand : 0;
  Sub* ibest = reinterpret_cast<Sub*>(route_smem);
  double* c_risk = reinterpret_cast<double*>(ibest + A.n_items);
  long long* c_cost = reinterpret_cast<long long*>(c_risk + n_cache);
  int* ch = reinterpret_cast<int*>(c_cost + n_cache);
  __shared__ long long wsum[32];
  __shared__ long long sh_total;
  __shared__ int sh_feasible, sh_fallback;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_pairs = A.n_items * A.n_cand;
  const bool cached = n_cache > 0;
  if (cached) {
    for (int p = tid; p < n_pairs; p += kThreads) {
      const int it = p / A.n_cand, k = p - it * A.n_cand;
      c_risk[p] = risk_of(A, it, k);
      c_cost[p] = cost_of(A, it, k);
    }
  }
  auto riskf = [&](int it, int k) -> double { return cached ? c_risk[it * A.n_cand + k] : risk_of(A, it, k); };
  auto costf = [&](int it, int k) -> long long { return cached ? c_cost[it * A.n_cand + k] : cost_of(A, it, k); };

  if (tid == 0) { sh_feasible = 1; sh_fallback = 0; }
  __syncthreads();
  if (A.prm.fixed_choice != nullptr) {
    for (int it = tid; it < A.n_items; it += kThreads) ch[it] = A.prm.fixed_choice[it];
    __syncthreads();
  } else {
    const bool global_pattern = A.prm.global_pattern != 0;
    if (global_pattern) {
      // Layer-level comparison router: every item takes the same candidate.  Lane c of warp 0 sums candidate c's cost
      // and risk over the items (risk in item order, one rounding per addition); the feasible candidate with the
      // smallest risk wins (ties: cheaper, lower index), else the cheapest one and the result is marked infeasible.
      if (warp == 0) {
        int b_inf = 2, b_c = -1;
        double b_risk = 0.0;
        long long b_cost = 0;
        for (int c = lane; c < A.n_cand; c += 32) {
          long long tot = A.prm.t_probe;
          double risk = 0.0;
          for (int it = 0; it < A.n_items; ++it) {
            tot += costf(it, c);
            risk = __dadd_rn(risk, riskf(it, c));
          }
          const int inf = tot <= A.prm.budget ? 0 : 1;
          if (inf) risk = 0.0;
          const bool take = b_c < 0 || inf < b_inf || (inf == b_inf && (risk < b_risk || (risk == b_risk && tot < b_cost)));
          if (take) { b_inf = inf; b_risk = risk; b_cost = tot; b_c = c; }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const int o_inf = __shfl_xor_sync(0xffffffffu, b_inf, off), o_c = __shfl_xor_sync(0xffffffffu, b_c, off);
          const double o_risk = __shfl_xor_sync(0xffffffffu, b_risk, off);
          const long long o_cost = __shfl_xor_sync(0xffffffffu, b_cost, off);
          bool take = false;
          if (o_c >= 0) {
            if (b_c < 0) take = true;
            else if (o_inf != b_inf) take = o_inf < b_inf;
            else if (o_risk != b_risk) take = o_risk < b_risk;
            else if (o_cost != b_cost) take = o_cost < b_cost;
            else take = o_c < b_c;
          }
          if (take) { b_inf = o_inf; b_risk = o_risk; b_cost = o_cost; b_c = o_c; }
        }
        for (int it = lane; it < A.n_items; it += 32) ch[it] = b_c;
        if (lane == 0) { sh_total = b_cost; sh_feasible = b_inf ? 0 : 1; }
      }
      __syncthreads();
    }
    if (!global_pattern) {
    for (int it = tid; it < A.n_items; it += kThreads) ch[it] = A.dense_c;
    long long part = 0;
    for (int it = tid; it < A.n_items; it += kThreads) part += costf(it, A.dense_c);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
    if (lane == 0) wsum[warp] = part;
    __syncthreads();
    if (tid == 0) {
      long long t = A.prm.t_probe;
      for (int w = 0; w < 32; ++w) t += wsum[w];
      sh_total = t;
    }
    __syncthreads();
    // ---- greedy substitutions until the layer budget is met.  Every item keeps its best substitution in shared
    // memory; a step only changes one item, so one warp finds the arg-min over items, applies it and refreshes that
    // item's entry without any block-wide barrier.
    auto best_of_item = [&](int it, int lane_k0, int stride) -> Sub {
      Sub best; best.ratio = 0.0; best.dT = 0; best.item = -1; best.k = -1;
      const int cur = ch[it];
      for (int k = lane_k0; k < A.n_cand; k += stride) {
        const long long dT = costf(it, cur) - costf(it, k);
        if (dT <= 0) continue;
        Sub s;
        s.ratio = __ddiv_rn(__dsub_rn(riskf(it, k), riskf(it, cur)), (double)dT);
        s.dT = dT; s.item = it; s.k = k;
        if (better(s, best)) best = s;
      }
      return best;
    };
    // An item's sequence of substitutions depends on that item alone, so when the tables fit in shared memory every
    // item's whole sequence is worked out first, one thread per item (that is where the divisions are); the serial part
    // is then a merge: take the best head of all sequences, pop it, until the budget is met.
    Sub* queue = reinterpret_cast<Sub*>(ch + A.n_items + (A.n_items & 1));      // [n_items][n_cand], 8-byte aligned
    int* qpos = reinterpret_cast<int*>(queue + (cached ? n_pairs : 0));         // [n_items] next entry, [n_items] length
    int* qlen = qpos + A.n_items;
    const bool sorted_path = cached && n_pairs <= kSortPairs;
    uint32_t* sidx = reinterpret_cast<uint32_t*>(qlen + A.n_items);             // [2048] (item << 8 | position), sorted
    unsigned char* mrun = reinterpret_cast<unsigned char*>(sidx + (sorted_path ? kSortPairs : 0));   // [n_pairs]
    if (cached) {
      for (int it = tid; it < A.n_items; it += kThreads) {
        int cur = A.dense_c, len = 0, m_at = 0;
        for (int guard = 0; guard < A.n_cand; ++guard) {
          Sub best; best.ratio = 0.0; best.dT = 0; best.item = -1; best.k = -1;
          for (int k = 0; k < A.n_cand; ++k) {
            const long long dT = costf(it, cur) - costf(it, k);
            if (dT <= 0) continue;
            Sub s2;
            s2.ratio = __ddiv_rn(__dsub_rn(riskf(it, k), riskf(it, cur)), (double)dT);
            s2.dT = dT; s2.item = it; s2.k = k;
            if (better(s2, best)) best = s2;
          }
          if (best.k < 0) break;
          queue[it * A.n_cand + len] = best;
          if (sorted_path) {                    // position of the largest key so far: an entry cannot be taken before it
            if (len == 0 || better(queue[it * A.n_cand + m_at], best)) m_at = len;
            mrun[it * A.n_cand + len] = (unsigned char)m_at;
          }
          ++len;
          cur = best.k;
        }
        qpos[it] = 0;
        qlen[it] = len;
      }
    } else {
      for (int it = tid; it < A.n_items; it += kThreads) ibest[it] = best_of_item(it, 0, 1);
    }
    __syncthreads();
    if (sorted_path) {
      // The merge takes, at every step, the smallest head.  An entry whose key is smaller than an earlier key of its own
      // sequence is taken right after that earlier entry, so the merged order is the order of the running maxima of
      // the keys (entries of one item by position): a sort, then one walk until the budget is met.
      __shared__ int sh_entries;
      if (tid == 0) {
        int acc = 0;
        for (int it = 0; it < A.n_items; ++it) { qpos[it] = acc; acc += qlen[it]; }
        sh_entries = acc;
      }
      __syncthreads();
      const int n_entries = sh_entries;
      int n_pad = 1;
      while (n_pad < n_entries) n_pad <<= 1;
      for (int x = tid; x < n_pad; x += kThreads) sidx[x] = 0xffffffffu;
      __syncthreads();
      for (int it = tid; it < A.n_items; it += kThreads)
        for (int j = 0; j < qlen[it]; ++j) sidx[qpos[it] + j] = ((uint32_t)it << 8) | (uint32_t)j;
      __syncthreads();
      auto before = [&](uint32_t a, uint32_t b) -> bool {        // a strictly before b in the merged order
        if (a == 0xffffffffu) return false;
        if (b == 0xffffffffu) return true;
        const int ia = (int)(a >> 8), ja = (int)(a & 255u), ib = (int)(b >> 8), jb = (int)(b & 255u);
        if (ia == ib) return ja < jb;
        return better(queue[ia * A.n_cand + mrun[ia * A.n_cand + ja]], queue[ib * A.n_cand + mrun[ib * A.n_cand + jb]]);
      };
      for (int k2 = 2; k2 <= n_pad; k2 <<= 1) {
        for (int j2 = k2 >> 1; j2 > 0; j2 >>= 1) {
          for (int x = tid; x < n_pad; x += kThreads) {
            const int y = x ^ j2;
            if (y > x) {
              const uint32_t a = sidx[x], b = sidx[y];
              const bool up = (x & k2) == 0;
              if (up ? before(b, a) : before(a, b)) { sidx[x] = b; sidx[y] = a; }
            }
          }
          __syncthreads();
        }
      }
      if (tid == 0) {
        long long total = sh_total;
        int x = 0;
        for (; x < n_entries && total > A.prm.budget; ++x) {
          const Sub e = queue[(sidx[x] >> 8) * A.n_cand + (sidx[x] & 255u)];
          ch[e.item] = e.k;
          total -= e.dT;
        }
        if (total > A.prm.budget) sh_feasible = 0;
        sh_total = total;
      }
      __syncthreads();
    }
    if (warp == 0) {
      long long total = sh_total;
      const int max_steps = n_pairs + 1;
      if (cached && !sorted_path) {
        for (int step = 0; step < max_steps && total > A.prm.budget; ++step) {
          Sub best; best.ratio = 0.0; best.dT = 0; best.item = -1; best.k = -1;
          for (int it = lane; it < A.n_items; it += 32) {
            const int qp = qpos[it];
            if (qp < qlen[it]) {
              const Sub s2 = queue[it * A.n_cand + qp];
              if (better(s2, best)) best = s2;
            }
          }
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
            const Sub o = shfl_sub(best, off);
            if (better(o, best)) best = o;
          }
          if (best.k < 0) { if (lane == 0) sh_feasible = 0; break; }
          if (lane == 0) { ch[best.item] = best.k; qpos[best.item] += 1; }
          total -= best.dT;
          __syncwarp();
        }
      }
      for (int step = 0; !cached && step < max_steps && total > A.prm.budget; ++step) {
        Sub best; best.ratio = 0.0; best.dT = 0; best.item = -1; best.k = -1;
        for (int it = lane; it < A.n_items; it += 32) {
          const Sub s = ibest[it];
          if (better(s, best)) best = s;
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const Sub o = shfl_sub(best, off);
          if (better(o, best)) best = o;
        }
        if (best.k < 0) { if (lane == 0) sh_feasible = 0; break; }
        if (lane == 0) ch[best.item] = best.k;
        total -= best.dT;
        __syncwarp();
        Sub mine = best_of_item(best.item, lane, 32);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const Sub o = shfl_sub(mine, off);
          if (better(o, mine)) mine = o;
        }
        if (lane == 0) ibest[best.item] = mine;
        __syncwarp();
      }
      // ---- back-fill: what is left of the budget goes to the substitutions with the largest risk decrease per unit
      // of added cost that still fit (ties: cheaper, lower item, lower candidate)
      if (A.prm.backfill != 0 && total <= A.prm.budget) {
        for (int step = 0; step < max_steps; ++step) {
          const long long slack = A.prm.budget - total;
          Sub best; best.ratio = 0.0; best.dT = 0; best.item = -1; best.k = -1;
          auto better_up = [](const Sub& a, const Sub& b) -> bool {
            if (a.k < 0) return false;
            if (b.k < 0) return true;
            if (a.ratio != b.ratio) return a.ratio < b.ratio;
            if (a.dT != b.dT) return a.dT < b.dT;
            if (a.item != b.item) return a.item < b.item;
            return a.k < b.k;
          };
          for (int it = lane; it < A.n_items; it += 32) {
            const int cur = ch[it];
            for (int k = 0; k < A.n_cand; ++k) {
              const long long dT = costf(it, k) - costf(it, cur);
              if (dT <= 0 || dT > slack) continue;
              const double dR = __dsub_rn(riskf(it, k), riskf(it, cur));
              if (!(dR < 0.0)) continue;
              Sub s2; s2.ratio = __ddiv_rn(dR, (double)dT); s2.dT = dT; s2.item = it; s2.k = k;
              if (better_up(s2, best)) best = s2;
            }
          }
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
            const Sub o = shfl_sub(best, off);
            if (better_up(o, best)) best = o;
          }
          if (best.k < 0) break;
          if (lane == 0) ch[best.item] = best.k;
          total += best.dT;
          __syncwarp();
        }
      }
      if (lane == 0) sh_total = total;
    }
    __syncthreads();
    }   // !global_pattern
    // ---- fallback walk: larger budget of the family first, then dense
    if (A.prm.use_cert) {
      for (int it = tid; it < A.n_items; it += kThreads) {
        const int s = it / A.Hq, h = it - s * A.Hq;
        const double vm = (double)A.vmax[s * A.Hkv + h / A.group];
        int c = ch[it];
        bool fired = false;
        for (int guard = 0; guard < RS_MAX_CANDIDATES + 1 && A.lib[c].pattern != RS_DENSE; ++guard) {
          const double m_low = fmax(0.0, __dsub_rn(m_hat_of(A, it, c), A.prm.delta_q));
          double cert = __dmul_rn(2.0, __dsub_rn(1.0, m_low));
          if (A.prm.cert_mode == RS_CERT_ABS) cert = __dmul_rn(cert, vm);
          if (!(cert > A.prm.cert_max)) break;
          fired = true;
          int nxt = A.prm.expand_first ? A.next_larger[c] : -1;
          if (nxt < 0 && A.prm.rescue_any != 0) {
            // rescue: the cheapest sparse candidate of any family whose certificate passes (ties: lower index)
            for (int k = 0; k < A.n_cand; ++k) {
              if (A.lib[k].pattern == RS_DENSE) continue;
              const double mk = fmax(0.0, __dsub_rn(m_hat_of(A, it, k), A.prm.delta_q));
              double ck = __dmul_rn(2.0, __dsub_rn(1.0, mk));
              if (A.prm.cert_mode == RS_CERT_ABS) ck = __dmul_rn(ck, vm);
              if (!(ck > A.prm.cert_max) && (nxt < 0 || costf(it, k) < costf(it, nxt))) nxt = k;
            }
          }
          c = (nxt >= 0) ? nxt : A.dense_c;
        }
        ch[it] = c;
        if (fired) atomicAdd(&sh_fallback, 1);
      }
      __syncthreads();
    }
  }
  if (A.prm.forced_dense != nullptr) {
    for (int it = tid; it < A.n_items; it += kThreads)
      if (A.prm.forced_dense[it] != 0) ch[it] = A.dense_c;
  }
  __syncthreads();
  for (int it = tid; it < A.n_items; it += kThreads) A.choice[it] = ch[it];
  if (A.report != nullptr) {
    long long part = 0;
    for (int it = tid; it < A.n_items; it += kThreads) part += cost_of(A, it, ch[it]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
    if (lane == 0) wsum[warp] = part;
    __syncthreads();
    if (tid == 0) {
      long long t = A.prm.t_probe;
      for (int w = 0; w < 32; ++w) t += wsum[w];
      double risk = 0.0;
      for (int it = 0; it < A.n_items; ++it) risk = __dadd_rn(risk, risk_of(A, it, ch[it]));
      A.report->total_cost = t;
      A.report->total_risk = risk;
      A.report->n_fallback = sh_fallback;
      A.report->feasible = sh_feasible;
    }
  }
  if (tid == 0 && sh_feasible == 0 && A.status != nullptr) A.status[3] = 1;   // budget cannot be met
}

}  // namespace

extern "C" int rs_route(const rs_problem* p, const rs_candidate* lib, int n_cand, const rs_cand_stats* stats,
                        const int64_t* cost, const float* vmax, const rs_route_params* params, int32_t* choice,
                        rs_route_report* report, int32_t* status, void* stream_) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!lib || n_cand <= 0 || n_cand > RS_MAX_CANDIDATES || !params || !choice) return RS_ERR_INVALID_ARG;
  const int n_items = p->n_segments * p->n_q_heads;
  if (n_items > kMaxItems) return RS_ERR_UNSUPPORTED_SHAPE;
  RouteArgs A{};
  A.n_items = n_items; A.n_cand = n_cand; A.Hq = p->n_q_heads; A.Hkv = p->n_kv_heads;
  A.group = p->n_q_heads / p->n_kv_heads; A.dense_c = -1;
  for (int c = 0; c < n_cand; ++c) {
    A.lib[c] = lib[c];
    if (lib[c].pattern == RS_DENSE && A.dense_c < 0) A.dense_c = c;
    A.next_larger[c] = -1;
    for (int k = c + 1; k < n_cand; ++k)
      if (lib[k].pattern == lib[c].pattern) { A.next_larger[c] = k; break; }
  }
  if (A.dense_c < 0) return RS_ERR_INVALID_ARG;          // the library must contain the dense candidate
  if (params->fixed_choice == nullptr && stats == nullptr) return RS_ERR_INVALID_ARG;
  if (params->use_cert && params->cert_mode == RS_CERT_ABS && vmax == nullptr) return RS_ERR_INVALID_ARG;
  A.stats = stats; A.cost = cost; A.vmax = vmax; A.prm = *params; A.choice = choice; A.report = report;
  A.status = status;
  const int n_pairs = n_items * n_cand;
  const size_t smem = (size_t)n_items * (sizeof(Sub) + sizeof(int)) + (n_pairs <= kCachePairs ? (size_t)n_pairs * (16 + sizeof(Sub)) : 0) +
                      (size_t)n_items * 8 + 32 + (n_pairs <= kSortPairs ? (size_t)kSortPairs * 4 + n_pairs : 0);
  static rs_smem_attr route_attr;
  if (rs_ensure_dynamic_smem(route_attr, rs_route_kernel, 200 * 1024) != RS_OK) return RS_ERR_CUDA;
  rs_route_kernel<<<1, kThreads, smem, (cudaStream_t)stream_>>>(A);
  return cudaGetLastError() == cudaSuccess ? RS_OK : RS_ERR_CUDA;
}
