// Acceptance along the draft tree: Algorithm 1 (multi-round speculative sampling, App. A.2) applied at every
// node from the committed context down (Sec. 3.3), or the greedy rule (Preliminaries).
//
// One team of threads walks one tree: a warp when the vocabulary is small (many trees per launch), a whole
// CTA otherwise.  Every thread of the team carries the same walk state; the vocabulary-wide steps (residual
// mass after a rejection, the final inverse-CDF draw, the greedy argmax) are spread over the team and reduced
// with warp shuffles (plus one shared-memory hop for a CTA team).  All sums and scalars are fp64.
//
// After m rejections at a node the residual distribution is not stored: an element is recomputed from the
// target row, the m rejected candidates' draft rows and their m normalisers,
//   x <- p(v);  for each rejected candidate j in order:  x <- max(0, x - p^_j(v)) / Z_j,
// which is exactly the sequence of updates Algorithm 1 performs (rows are L2-resident after their first use).
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCtaTeam = 512;
constexpr int kWarpTeamsPerCta = 8;

template <int NT>
struct TeamScratch {
  double d[NT / 32 > 0 ? NT / 32 : 1];
  unsigned long long u[NT / 32 > 0 ? NT / 32 : 1];
};

template <int NT>
struct Team {
  int rank;
  TeamScratch<NT>* sc;

  __device__ __forceinline__ void sync() const {
    if (NT == 32) __syncwarp();
    else __syncthreads();
  }
  // Sum over the team; every thread gets the same value, combined in a fixed order.
  __device__ double sum(double v) const {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (NT == 32) return v;
    __syncthreads();
    if ((rank & 31) == 0) sc->d[rank >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += sc->d[w];
    return t;
  }
  __device__ unsigned long long max_u64(unsigned long long v) const {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long x = __shfl_xor_sync(0xffffffffu, v, o);
      v = x > v ? x : v;
    }
    if (NT == 32) return v;
    __syncthreads();
    if ((rank & 31) == 0) sc->u[rank >> 5] = v;
    __syncthreads();
    unsigned long long t = 0ull;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t = sc->u[w] > t ? sc->u[w] : t;
    return t;
  }
  // Exclusive prefix of v in rank order, and the team total.
  __device__ double exclusive_scan(double v, double* total) const {
    double inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double x = __shfl_up_sync(0xffffffffu, inc, o);
      if ((rank & 31) >= o) inc += x;
    }
    double before = 0.0;
    if (NT == 32) {
      *total = __shfl_sync(0xffffffffu, inc, 31);
    } else {
      __syncthreads();
      if ((rank & 31) == 31) sc->d[rank >> 5] = inc;
      __syncthreads();
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < NT / 32; ++w) {
        if (w == (rank >> 5)) before = t;
        t += sc->d[w];
      }
      *total = t;
    }
    const double prev = __shfl_up_sync(0xffffffffu, inc, 1);
    return before + ((rank & 31) ? prev : 0.0);
  }
};

__device__ __forceinline__ unsigned int ordered_bits(float f) {
  const unsigned int u = __float_as_uint(f + 0.0f);   // -0 becomes +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Chain {
  const float* target_row;
  const float* draft_base;  // draft rows of this sequence
  const int* rej;           // rejected candidates at the current node, in order
  const double* Z;          // their normalisers
  int n_rej;
  int V;
  // residual probability of token v after the rejections recorded so far
  __device__ __forceinline__ double at(int v) const {
    double x = static_cast<double>(target_row[v]);
    for (int j = 0; j < n_rej; ++j) {
      const double d = x - static_cast<double>(draft_base[static_cast<size_t>(rej[j]) * V + v]);
      x = (d > 0.0 ? d : 0.0) / Z[j];
    }
    return x;
  }
};

template <int NT>
__global__ void __launch_bounds__(NT == 32 ? 32 * kWarpTeamsPerCta : NT) accept_kernel(AcceptParams p) {
  constexpr int TEAMS = NT == 32 ? kWarpTeamsPerCta : 1;
  __shared__ TeamScratch<NT> s_scratch[TEAMS];
  __shared__ int s_par[TEAMS][kMaxTree], s_tok[TEAMS][kMaxTree], s_rej[TEAMS][kMaxTree];
  __shared__ double s_Z[TEAMS][kMaxTree];

  const int team_id = NT == 32 ? (threadIdx.x >> 5) : 0;
  const int b = NT == 32 ? blockIdx.x * TEAMS + team_id : blockIdx.x;
  if (b >= p.B) return;   // a whole team leaves together (a warp, or the CTA)
  Team<NT> team;
  team.rank = NT == 32 ? (threadIdx.x & 31) : threadIdx.x;
  team.sc = &s_scratch[team_id];
  int* par = s_par[team_id];
  int* tok = s_tok[team_id];
  int* rej = s_rej[team_id];
  double* Zs = s_Z[team_id];

  const int T = p.T, V = p.V;
  int n = p.tree_sizes ? p.tree_sizes[b] : T;
  const bool is_greedy = p.greedy && p.greedy[b] != 0;
  int bad = (n < 0 || n > T) ? EAGLE_ERR_TREE : 0;
  if (!bad && !is_greedy && (!p.draft || !p.uniforms)) bad = EAGLE_ERR_NULL;  // a stochastic walk needs both
  if (bad) n = 0;
  for (int i = team.rank; i < n; i += NT) {
    const int pi = p.parent[static_cast<size_t>(b) * T + i];
    const int ti = p.tokens[static_cast<size_t>(b) * T + i];
    par[i] = pi;
    tok[i] = ti;
  }
  team.sync();
  if (!bad) {
    // every thread checks every node, so the verdict is the same everywhere
    for (int i = 0; i < n; ++i) {
      if (par[i] < -1 || par[i] >= i) bad = EAGLE_ERR_TREE;
      else if (tok[i] < 0 || tok[i] >= V) bad = bad ? bad : EAGLE_ERR_TOKEN;
    }
  }
  int32_t* path = p.path + static_cast<size_t>(b) * p.path_cap;
  for (int j = team.rank; j < p.path_cap; j += NT) path[j] = -1;
  if (bad) {
    if (team.rank == 0) {
      report_status(p.status, bad);
      p.bonus[b] = -1;
      if (p.accept_len) p.accept_len[b] = 0;
    }
    return;
  }
  team.sync();   // the -1 fill is ordered before the path entries written below (same team)

  const float* target_b = p.target + static_cast<size_t>(b) * (T + 1) * V;
  const float* draft_b = p.draft ? p.draft + static_cast<size_t>(b) * T * V : nullptr;
  const float* uni_b = p.uniforms ? p.uniforms + static_cast<size_t>(b) * (T + 1) : nullptr;

  int cur = -1, len = 0, bonus = -1;
  for (;;) {
    const float* prow = target_b + static_cast<size_t>(cur + 1) * V;
    int next = -1;
    if (is_greedy) {
      // argmax, lowest token id on ties: key = (ordered value, ~id)
      unsigned long long best = 0ull;
      for (int v = team.rank; v < V; v += NT) {
        const unsigned long long key = (static_cast<unsigned long long>(ordered_bits(prow[v])) << 32) |
                                       static_cast<unsigned int>(~static_cast<unsigned int>(v));
        best = key > best ? key : best;
      }
      best = team.max_u64(best);
      const int a = static_cast<int>(~static_cast<unsigned int>(best & 0xffffffffull));
      for (int i = 0; i < n && next < 0; ++i)
        if (par[i] == cur && tok[i] == a) next = i;
      if (next < 0) bonus = a;
    } else {
      Chain ch{prow, draft_b, rej, Zs, 0, V};
      for (int i = 0; i < n && next < 0; ++i) {
        if (par[i] != cur) continue;
        const float* qrow = draft_b + static_cast<size_t>(i) * V;
        const int t = tok[i];
        const double r = static_cast<double>(uni_b[i]);
        const double pt = ch.at(t), qt = static_cast<double>(qrow[t]);
        if (r * qt < pt) {
          next = i;
        } else {
          // mass of max(0, p - p^_i) over the vocabulary
          double z = 0.0;
          for (int v = team.rank; v < V; v += NT) {
            const double d = ch.at(v) - static_cast<double>(qrow[v]);
            z += d > 0.0 ? d : 0.0;
          }
          z = team.sum(z);
          if (z > 0.0) {           // zero residual mass: the distribution is kept as it is
            team.sync();           // nobody still reads the list with the old length
            if (team.rank == 0) {
              rej[ch.n_rej] = i;
              Zs[ch.n_rej] = z;
            }
            team.sync();
            ch.n_rej += 1;
          }
        }
      }
      if (next < 0) {
        // inverse CDF in ascending token id: contiguous chunk per thread, scan of chunk sums, rescan of one chunk
        const double u = static_cast<double>(uni_b[T]);
        const int chunk = (V + NT - 1) / NT;
        const int v0 = team.rank * chunk < V ? team.rank * chunk : V;
        const int v1 = v0 + chunk < V ? v0 + chunk : V;
        double s = 0.0;
        int last_pos = -1;
        for (int v = v0; v < v1; ++v) {
          const double x = ch.at(v);
          if (x > 0.0) last_pos = v;
          s += x;
        }
        double total;
        const double before = team.exclusive_scan(s, &total);
        const double thr = u * total;
        const bool mine = before + s > thr;
        // first thread (lowest rank) whose inclusive prefix passes the threshold; else the last positive token
        const unsigned long long key_owner = mine ? (0x100000000ull | static_cast<unsigned int>(~static_cast<unsigned int>(team.rank))) : 0ull;
        const unsigned long long key_last = static_cast<unsigned long long>(static_cast<unsigned int>(last_pos + 1));
        const unsigned long long w_owner = team.max_u64(key_owner);
        int x_found = -1;
        if (w_owner) {
          const int owner = static_cast<int>(~static_cast<unsigned int>(w_owner & 0xffffffffull));
          unsigned long long key_x = 0ull;
          if (team.rank == owner) {
            double c = 0.0;
            for (int v = v0; v < v1; ++v) {
              c += ch.at(v);
              if (before + c > thr) {
                key_x = static_cast<unsigned long long>(v) + 1ull;
                break;
              }
            }
          }
          x_found = static_cast<int>(team.max_u64(key_x)) - 1;
        }
        if (x_found < 0) {
          const int lp = static_cast<int>(team.max_u64(key_last)) - 1;
          x_found = lp >= 0 ? lp : V - 1;
        }
        bonus = x_found;
      }
    }
    if (next < 0) break;
    if (team.rank == 0 && len < p.path_cap) path[len] = next;
    ++len;
    cur = next;
    team.sync();   // the rejected-candidate list of the finished node is dead before the next node reuses it
  }
  if (team.rank == 0) {
    p.bonus[b] = bonus;
    if (p.accept_len) p.accept_len[b] = len;
  }
}

}  // namespace

cudaError_t launch_accept(const AcceptParams& p, cudaStream_t stream) {
  if (p.B == 0) return cudaSuccess;
  if (p.V <= 4096) {
    const unsigned blocks = static_cast<unsigned>((p.B + kWarpTeamsPerCta - 1) / kWarpTeamsPerCta);
    accept_kernel<32><<<blocks, 32 * kWarpTeamsPerCta, 0, stream>>>(p);
  } else {
    accept_kernel<kCtaTeam><<<static_cast<unsigned>(p.B), kCtaTeam, 0, stream>>>(p);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
