// Acceptance along the draft tree: Algorithm 1 (multi-round speculative sampling, App. A.2) applied at every
// node from the committed context down (Sec. 3.3), or the greedy rule (Preliminaries).
//
// One team of threads walks one tree; every thread of the team carries the same walk state, and the
// vocabulary-wide steps (residual mass after a rejection, the final inverse-CDF draw, the greedy argmax) are
// spread over the team.  A team is
//   - one warp when the vocabulary is small (many trees per CTA), or
//   - a thread-block cluster of 1, 2, 4 or 8 CTAs of 512 threads (fewer trees -> wider teams, so that one
//     tree's 128 KB rows are pulled by several SMs at once); partial results cross CTAs through
//     distributed shared memory and a cluster barrier.
// Thread g of a team owns the contiguous token range [g*chunk, (g+1)*chunk) in every sweep, so prefix sums in
// token order need one scan of per-thread sums.  All sums and scalars are fp64; reductions combine partials
// in a fixed order, so a call is reproducible bit for bit.
//
// After m rejections at a node the residual is not stored but recomputed, unnormalised, from the target row,
// the rejected candidates' draft rows and m scalars:  u_0 = p, W_0 = 1,
//   u_k(v) = max(0, u_{k-1}(v) - W_{k-1} * p^_k(v)),   W_k = sum_v u_k(v),
// so that Algorithm 1's normalised residual is u_m / W_m, its accept test r < p(t)/p^(t) reads
// r * p^(t) * W_m < u_m(t), and the final draw (scale-free) is taken from u_m.  No division is needed.
//
// Logits instead of probabilities (LOGITS = true): a row is softmax(z / T), never materialised.  Each row the walk
// touches costs one more sweep for its maximum m and its mass Z = sum_v w(v), w(v) = 2^((z_v - m) * log2(e) / T);
// then u_0 = w of the target row with W_0 = Z, and a draft row enters as p^ = w^ / Z^ (the scalar 1 / Z^ is folded
// into the stored W_k).  Exponentials are fp32 (the logits are), sums fp64.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCtaThreads = 512;
constexpr int kWarpTeamsPerCta = 8;
constexpr int kMaxCluster = 8;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void dsmem_store_u64(const void* local_smem, uint32_t cta, unsigned long long v) {
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(local_smem));
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(cta));
  asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(ra), "l"(v) : "memory");
}

// NT threads per CTA (32: a warp is the team), CL CTAs per team.
template <int NT, int CL>
struct Team {
  static constexpr int kWarps = NT / 32;
  struct Scratch {
    unsigned long long warp[kWarps > 0 ? kWarps : 1];
    unsigned long long xch[2][kMaxCluster];   // all-gather slots, double buffered
  };
  Scratch* sc;
  int tid;        // thread within the CTA (or lane, for a warp team)
  int cta;        // CTA rank within the cluster
  int phase;      // which xch buffer the next cross-CTA exchange uses

  __device__ __forceinline__ int rank() const { return cta * NT + tid; }
  static constexpr int kSize = NT * CL;

  __device__ __forceinline__ void sync_cta() const {
    if (NT == 32) __syncwarp();
    else __syncthreads();
  }
  // every CTA publishes one 64-bit word to all CTAs; afterwards xch[buf][c] holds CTA c's word everywhere
  __device__ __forceinline__ int exchange(unsigned long long mine) {
    const int buf = phase;
    phase ^= 1;
    if (tid < CL) dsmem_store_u64(&sc->xch[buf][cta], static_cast<uint32_t>(tid), mine);
    cluster_sync_all();
    return buf;
  }
  __device__ double sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (NT == 32) return v;
    __syncthreads();
    if ((tid & 31) == 0) sc->warp[tid >> 5] = __double_as_longlong(v);
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += __longlong_as_double(sc->warp[w]);
    if (CL == 1) return t;
    const int buf = exchange(__double_as_longlong(t));
    double a = 0.0;
#pragma unroll
    for (int c = 0; c < CL; ++c) a += __longlong_as_double(sc->xch[buf][c]);
    return a;
  }
  __device__ unsigned long long max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long x = __shfl_xor_sync(0xffffffffu, v, o);
      v = x > v ? x : v;
    }
    if (NT == 32) return v;
    __syncthreads();
    if ((tid & 31) == 0) sc->warp[tid >> 5] = v;
    __syncthreads();
    unsigned long long t = 0ull;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t = sc->warp[w] > t ? sc->warp[w] : t;
    if (CL == 1) return t;
    const int buf = exchange(t);
    unsigned long long a = 0ull;
#pragma unroll
    for (int c = 0; c < CL; ++c) a = sc->xch[buf][c] > a ? sc->xch[buf][c] : a;
    return a;
  }
  // exclusive prefix of v in team-rank order, and the team total
  __device__ double exclusive_scan(double v, double* total) {
    double inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double x = __shfl_up_sync(0xffffffffu, inc, o);
      if ((tid & 31) >= o) inc += x;
    }
    const double prev = __shfl_up_sync(0xffffffffu, inc, 1);
    double before = (tid & 31) ? prev : 0.0;
    if (NT == 32) {
      *total = __shfl_sync(0xffffffffu, inc, 31);
      return before;
    }
    __syncthreads();
    if ((tid & 31) == 31) sc->warp[tid >> 5] = __double_as_longlong(inc);
    __syncthreads();
    double t = 0.0, warp_before = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      if (w == (tid >> 5)) warp_before = t;
      t += __longlong_as_double(sc->warp[w]);
    }
    before = warp_before + before;
    if (CL == 1) {
      *total = t;
      return before;
    }
    const int buf = exchange(__double_as_longlong(t));
    double a = 0.0, cta_before = 0.0;
#pragma unroll
    for (int c = 0; c < CL; ++c) {
      if (c == cta) cta_before = a;
      a += __longlong_as_double(sc->xch[buf][c]);
    }
    *total = a;
    return cta_before + before;
  }
};

__device__ __forceinline__ unsigned int ordered_bits(float f) {
  const unsigned int u = __float_as_uint(f + 0.0f);   // -0 becomes +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float from_ordered_bits(unsigned int b) {
  return __uint_as_float((b & 0x80000000u) ? (b & 0x7fffffffu) : ~b);
}

// The residual after the rejections recorded so far, evaluated on the fly.
template <bool LOGITS>
struct Residual {
  const float* target_row;
  const float* draft_base;  // draft rows of this sequence
  const int* rej;           // rejected candidates at the current node, in order
  const double* scale;      // scale[k] = W_k, the mass of the residual before rejection k+1 (W_0 = 1); logits: W_k / Z^_k
  const float* row_max;     // logits: maximum of the rejected candidates' draft rows
  float t_max, c;           // logits: maximum of the target row; log2(e) / temperature
  int m;                    // rejections recorded
  int V;

  // value of a row entry: the probability as given, or the unnormalised softmax weight
  __device__ __forceinline__ double val(float z, float zmax) const {
    if (LOGITS) return static_cast<double>(exp2f((z - zmax) * c));
    return static_cast<double>(z);
  }
  __device__ __forceinline__ double at(int v) const {
    double x = val(__ldg(target_row + v), t_max);
    for (int k = 0; k < m; ++k)
      x = fmax(0.0, fma(-scale[k], val(__ldg(draft_base + static_cast<size_t>(rej[k]) * V + v), LOGITS ? row_max[k] : 0.f), x));
    return x;
  }
  // four consecutive tokens starting at v (v % 4 == 0, rows 16-byte aligned)
  __device__ __forceinline__ void at4(int v, double (&x)[4]) const {
    const float4 t = __ldg(reinterpret_cast<const float4*>(target_row + v));
    x[0] = val(t.x, t_max); x[1] = val(t.y, t_max); x[2] = val(t.z, t_max); x[3] = val(t.w, t_max);
    for (int k = 0; k < m; ++k) {
      const float4 q = __ldg(reinterpret_cast<const float4*>(draft_base + static_cast<size_t>(rej[k]) * V + v));
      const double w = -scale[k];
      const float qm = LOGITS ? row_max[k] : 0.f;
      x[0] = fmax(0.0, fma(w, val(q.x, qm), x[0]));
      x[1] = fmax(0.0, fma(w, val(q.y, qm), x[1]));
      x[2] = fmax(0.0, fma(w, val(q.z, qm), x[2]));
      x[3] = fmax(0.0, fma(w, val(q.w, qm), x[3]));
    }
  }
};

struct TreeSmem {
  int par[kMaxTree], tok[kMaxTree], rej[kMaxTree];
  double scale[kMaxTree];
  float row_max[kMaxTree];
};

template <int NT, int CL, bool LOGITS>
__global__ void __launch_bounds__(NT == 32 ? 32 * kWarpTeamsPerCta : NT) accept_kernel(AcceptParams p) {
  using TeamT = Team<NT, CL>;
  constexpr int TEAMS = NT == 32 ? kWarpTeamsPerCta : 1;
  __shared__ typename TeamT::Scratch s_scratch[TEAMS];
  __shared__ TreeSmem s_tree[TEAMS];

  const int team_id = NT == 32 ? (threadIdx.x >> 5) : 0;
  TeamT team;
  team.tid = NT == 32 ? (threadIdx.x & 31) : threadIdx.x;
  team.cta = CL > 1 ? static_cast<int>(cluster_ctarank()) : 0;
  team.phase = 0;
  team.sc = &s_scratch[team_id];
  const int b = NT == 32 ? blockIdx.x * TEAMS + team_id : static_cast<int>(blockIdx.x) / CL;
  if (b >= p.B) return;   // a whole team leaves together (a warp; clusters are launched exactly)
  TreeSmem& ts = s_tree[team_id];

  const int T = p.T, V = p.V;
  const int tb = p.shared_tree ? 0 : b;   // one tree for every sequence, or one per sequence
  int n = p.tree_sizes ? p.tree_sizes[tb] : T;
  const bool is_greedy = p.greedy && p.greedy[b] != 0;
  int bad = (n < 0 || n > T) ? EAGLE_ERR_TREE : 0;
  if (!bad && !is_greedy && (!p.draft || !p.uniforms)) bad = EAGLE_ERR_NULL;  // a stochastic walk needs both
  if (bad) n = 0;
  for (int i = team.tid; i < n; i += NT) {
    ts.par[i] = p.parent[static_cast<size_t>(tb) * T + i];
    ts.tok[i] = p.tokens[static_cast<size_t>(b) * T + i];
  }
  team.sync_cta();
  if (!bad) {
    // every thread checks every node, so the verdict is the same everywhere
    for (int i = 0; i < n; ++i) {
      if (ts.par[i] < -1 || ts.par[i] >= i) bad = EAGLE_ERR_TREE;
      else if (ts.tok[i] < 0 || ts.tok[i] >= V) bad = bad ? bad : EAGLE_ERR_TOKEN;
    }
  }
  const bool writer = team.rank() == 0;
  int32_t* path = p.path + static_cast<size_t>(b) * p.path_cap;
  if (team.cta == 0)
    for (int j = team.tid; j < p.path_cap; j += NT) path[j] = -1;
  if (bad) {
    if (writer) {
      report_status(p.status, bad);
      p.bonus[b] = -1;
      if (p.accept_len) p.accept_len[b] = 0;
    }
    return;   // uniform over the team: nobody is left waiting at a cluster barrier
  }
  team.sync_cta();   // the -1 fill is ordered before the path entries written below (same CTA)

  const float* target_b = p.target + static_cast<size_t>(b) * (T + 1) * V;
  const float* draft_b = p.draft ? p.draft + static_cast<size_t>(b) * T * V : nullptr;
  const float* uni_b = p.uniforms ? p.uniforms + static_cast<size_t>(b) * (T + 1) : nullptr;

  // token range of this thread; vector loads need V % 4 == 0 (then every row starts 16-byte aligned)
  const bool vec = (V & 3) == 0 && (reinterpret_cast<uintptr_t>(p.target) & 15) == 0 &&
                   (p.draft == nullptr || (reinterpret_cast<uintptr_t>(p.draft) & 15) == 0);
  int chunk = (V + TeamT::kSize - 1) / TeamT::kSize;
  chunk = (chunk + 3) & ~3;
  const int v0 = min(team.rank() * chunk, V), v1 = min(v0 + chunk, V);

  // logits: maximum and softmax mass of a row (two sweeps of the thread's range, the second from cache)
  const float c = p.inv_temp_log2;
  auto row_stats = [&](const float* row, float* zmax, double* mass) {
    float mx = -INFINITY;
    if (vec) {
#pragma unroll 4
      for (int v = v0; v < v1; v += 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(row + v));
        mx = fmaxf(fmaxf(mx, fmaxf(t.x, t.y)), fmaxf(t.z, t.w));
      }
    } else {
      for (int v = v0; v < v1; ++v) mx = fmaxf(mx, __ldg(row + v));
    }
    mx = from_ordered_bits(static_cast<unsigned int>(team.max_u64(static_cast<unsigned long long>(ordered_bits(mx)) << 32) >> 32));
    double z = 0.0;
    if (vec) {
#pragma unroll 4
      for (int v = v0; v < v1; v += 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(row + v));
        z += static_cast<double>(exp2f((t.x - mx) * c)) + static_cast<double>(exp2f((t.y - mx) * c));
        z += static_cast<double>(exp2f((t.z - mx) * c)) + static_cast<double>(exp2f((t.w - mx) * c));
      }
    } else {
      for (int v = v0; v < v1; ++v) z += static_cast<double>(exp2f((__ldg(row + v) - mx) * c));
    }
    *zmax = mx;
    *mass = team.sum(z);
  };

  int cur = -1, len = 0, bonus = -1;
  for (;;) {
    const float* prow = target_b + static_cast<size_t>(cur + 1) * V;
    int next = -1;
    if (is_greedy) {
      // argmax, lowest token id on ties: key = (ordered value, ~id)
      unsigned long long best = 0ull;
      auto consider = [&](float f, int v) {
        const unsigned long long key = (static_cast<unsigned long long>(ordered_bits(f)) << 32) | static_cast<unsigned int>(~static_cast<unsigned int>(v));
        best = key > best ? key : best;
      };
      if (vec) {
#pragma unroll 4
        for (int v = v0; v < v1; v += 4) {
          const float4 t = __ldg(reinterpret_cast<const float4*>(prow + v));
          consider(t.x, v); consider(t.y, v + 1); consider(t.z, v + 2); consider(t.w, v + 3);
        }
      } else {
        for (int v = v0; v < v1; ++v) consider(__ldg(prow + v), v);
      }
      best = team.max_u64(best);
      const int a = static_cast<int>(~static_cast<unsigned int>(best & 0xffffffffull));
      for (int i = 0; i < n && next < 0; ++i)
        if (ts.par[i] == cur && ts.tok[i] == a) next = i;
      if (next < 0) bonus = a;
    } else {
      Residual<LOGITS> res{prow, draft_b, ts.rej, ts.scale, ts.row_max, 0.f, c, 0, V};
      double W = 1.0;   // mass of the current residual
      if (LOGITS) row_stats(prow, &res.t_max, &W);
      for (int i = 0; i < n && next < 0; ++i) {
        if (ts.par[i] != cur) continue;
        const float* qrow = draft_b + static_cast<size_t>(i) * V;
        const int t = ts.tok[i];
        // If the candidate is rejected, this thread's part of its draft row (and, before the first rejection at this
        // node, of the target row) is swept next: ask for it now, together with the two scalars of the test, so that
        // the sweep does not start with a second trip to memory.
        if (v0 < v1) {
          asm volatile("prefetch.global.L1 [%0];" ::"l"(qrow + v0));
          if (res.m == 0) asm volatile("prefetch.global.L1 [%0];" ::"l"(prow + v0));
        }
        const double r = static_cast<double>(uni_b[i]);
        float q_max = 0.f;
        double q_inv = 1.0;     // 1 / mass of the candidate's draft row
        if (LOGITS) {
          double q_mass;
          row_stats(qrow, &q_max, &q_mass);
          q_inv = 1.0 / q_mass;
        }
        const double Wq = W * q_inv;   // what a draft-row entry is multiplied with inside the residual
        const double ut = res.at(t), qt = res.val(__ldg(qrow + t), q_max);
        if (r * qt * Wq < ut) {
          next = i;
        } else {
          // mass of max(0, u - W * p^_i) over the vocabulary
          double z = 0.0;
          if (vec) {
#pragma unroll 4
            for (int v = v0; v < v1; v += 4) {
              double x[4];
              res.at4(v, x);
              const float4 q = __ldg(reinterpret_cast<const float4*>(qrow + v));
              z += fmax(0.0, fma(-Wq, res.val(q.x, q_max), x[0]));
              z += fmax(0.0, fma(-Wq, res.val(q.y, q_max), x[1]));
              z += fmax(0.0, fma(-Wq, res.val(q.z, q_max), x[2]));
              z += fmax(0.0, fma(-Wq, res.val(q.w, q_max), x[3]));
            }
          } else {
            for (int v = v0; v < v1; ++v) z += fmax(0.0, fma(-Wq, res.val(__ldg(qrow + v), q_max), res.at(v)));
          }
          z = team.sum(z);
          if (z > 0.0) {           // zero residual mass: the distribution is kept as it is
            // entry res.m is not read by anyone yet (readers stop at res.m), so it can be written in place
            if (team.tid == 0) {
              ts.rej[res.m] = i;
              ts.scale[res.m] = Wq;
              ts.row_max[res.m] = q_max;
            }
            team.sync_cta();
            res.m += 1;
            W = z;
          }
        }
      }
      if (next < 0) {
        // final draw by inverse CDF over the residual, ascending token id: per-thread sums of contiguous
        // ranges, one scan, then the owning thread walks its own range
        const double u = static_cast<double>(uni_b[T]);
        double s = 0.0;
        int last_pos = -1;
        if (vec) {
#pragma unroll 4
          for (int v = v0; v < v1; v += 4) {
            double x[4];
            res.at4(v, x);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              s += x[e];
              if (x[e] > 0.0) last_pos = v + e;
            }
          }
        } else {
          for (int v = v0; v < v1; ++v) {
            const double x = res.at(v);
            s += x;
            if (x > 0.0) last_pos = v;
          }
        }
        double total;
        const double before = team.exclusive_scan(s, &total);
        const double thr = u * total;
        const bool mine = before + s > thr;
        // the first thread (lowest rank) whose inclusive prefix passes the threshold finds the token inside its
        // range by repeating exactly the additions that produced s
        unsigned long long key = 0ull;
        if (mine) {
          int x_found = v1 - 1;
          double c = 0.0;
          bool found = false;
          if (vec) {
            for (int v = v0; v < v1 && !found; v += 4) {
              double x[4];
              res.at4(v, x);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                c += x[e];
                if (!found && before + c > thr) {
                  x_found = v + e;
                  found = true;
                }
              }
            }
          } else {
            for (int v = v0; v < v1 && !found; ++v) {
              c += res.at(v);
              if (before + c > thr) {
                x_found = v;
                found = true;
              }
            }
          }
          // rank in the high half (inverted: lowest rank wins the max), token in the low half
          key = (static_cast<unsigned long long>(0x7fffffffu - static_cast<unsigned int>(team.rank())) << 32) |
                static_cast<unsigned int>(x_found + 1);
        }
        const unsigned long long win = team.max_u64(key);
        if (win) {
          bonus = static_cast<int>(win & 0xffffffffull) - 1;
        } else {
          // rounding left u * total at or above every prefix: take the last token with positive mass
          const int lp = static_cast<int>(team.max_u64(static_cast<unsigned long long>(static_cast<unsigned int>(last_pos + 1)))) - 1;
          bonus = lp >= 0 ? lp : V - 1;
        }
      }
    }
    if (next < 0) break;
    if (writer && len < p.path_cap) path[len] = next;
    ++len;
    cur = next;
    team.sync_cta();   // the rejected-candidate list of the finished node is dead before the next node reuses it
  }
  if (writer) {
    p.bonus[b] = bonus;
    if (p.accept_len) p.accept_len[b] = len;
  }
}

template <int CL>
cudaError_t launch_cluster(const AcceptParams& p, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(p.B) * CL, 1, 1);
  cfg.blockDim = dim3(kCtaThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.logits) return cudaLaunchKernelEx(&cfg, accept_kernel<kCtaThreads, CL, true>, p);
  return cudaLaunchKernelEx(&cfg, accept_kernel<kCtaThreads, CL, false>, p);
}

}  // namespace

// Team width: a warp per tree for small vocabularies (returned as 0); otherwise CTAs of 512 threads in clusters as
// wide as still fit the GPU with at most four CTAs per SM: the walk is a chain of dependent vocabulary sweeps, so a
// tree finishes sooner the more SMs pull its rows.  (With 64 registers per thread only two CTAs of 512 threads are
// resident per SM, so at batch 64 the clusters of eight run in two waves; measured, that is still faster than clusters
// of four in one wave: 52 against 57 us on the 64-sequence mix.)  A call that passes no draft rows or no uniforms has
// only greedy sequences (one argmax sweep per visited node, no rows to subtract): there clusters of four in one wave
// are the faster ones (35 against 46 us at batch 64), so that case takes four where eight would need a second wave.
int accept_cluster_width(int batch, int vocab, int sm_count, bool all_greedy) {
  if (vocab <= 4096) return 0;
  if (all_greedy && 8ll * batch > 2ll * sm_count && 4ll * batch <= 2ll * sm_count) return 4;
  const long long resident = 4ll * sm_count;
  if (8ll * batch <= resident) return 8;
  if (4ll * batch <= resident) return 4;
  if (2ll * batch <= resident) return 2;
  return 1;
}

cudaError_t launch_accept(const AcceptParams& p, int sm_count, cudaStream_t stream) {
  if (p.B == 0) return cudaSuccess;
  cudaError_t e;
  switch (accept_cluster_width(p.B, p.V, sm_count, p.draft == nullptr || p.uniforms == nullptr)) {
    case 0: {
      const unsigned blocks = static_cast<unsigned>((p.B + kWarpTeamsPerCta - 1) / kWarpTeamsPerCta);
      if (p.logits) accept_kernel<32, 1, true><<<blocks, 32 * kWarpTeamsPerCta, 0, stream>>>(p);
      else accept_kernel<32, 1, false><<<blocks, 32 * kWarpTeamsPerCta, 0, stream>>>(p);
      e = cudaGetLastError();
      break;
    }
    case 8: e = launch_cluster<8>(p, stream); break;
    case 4: e = launch_cluster<4>(p, stream); break;
    case 2: e = launch_cluster<2>(p, stream); break;
    default:
      if (p.logits) accept_kernel<kCtaThreads, 1, true><<<static_cast<unsigned>(p.B), kCtaThreads, 0, stream>>>(p);
      else accept_kernel<kCtaThreads, 1, false><<<static_cast<unsigned>(p.B), kCtaThreads, 0, stream>>>(p);
      e = cudaGetLastError();
  }
  count_launch();
  return e;
}

}  // namespace eagle
