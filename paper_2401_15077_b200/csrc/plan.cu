// Device-side planner of the tree-verification attention call, and the stand-alone tree-mask builder.
//
// The host never reads seq_lens or tree_sizes (they are device arrays and the call must not synchronise),
// so one small CTA turns them into (1) the per-node ancestor-or-self bit masks that define tree attention
// (Sec. 3.1 / 3.3: a draft token attends to the context and to its own root path) and (2) the work split of
// the persistent attention kernel.
//
// Work split.  A work unit is one 128-row query tile of one (sequence, KV head); its work is the sequence's KV
// tiles.  The CTAs of the attention kernel are taken in pairs ("teams").  The query tiles of a (sequence, KV head)
// are taken two at a time: such a pair is a super-unit that both CTAs of a team walk together, one query tile each
// over the same KV tiles, so the keys and values one of them pulls from HBM are still in L2 when the other asks for
// them; the odd last query tiles of two neighbouring KV heads form a twin super-unit (one head per CTA of the team,
// same KV range), and with an odd number of KV heads the last head's odd tile is a lone super-unit whose KV range the
// team's two CTAs split in halves.  All super-units
// are laid end to end on one line (plus `item_overhead_tiles` positions of fixed cost at the start of each), and
// every team gets an equal contiguous share of the line.  A share boundary inside a super-unit cuts it into
// pieces (their partial results are merged by the combine kernel); boundaries closer than `snap_tiles` to an edge
// move to the edge.  Every CTA therefore does the same number of KV tiles, to within the snap, whatever the mix of
// sequence lengths and tree sizes.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kPlanThreads = 1024;

// Two exclusive prefix sums at once, of value(i).a (64-bit) and value(i).b (32-bit), i in [0, n), by one CTA;
// put(i, prefix_a, prefix_b) stores them; returns the totals.
// Thread chunks -> warp scan -> scan of the 32 warp totals by the first warp -> back to the threads.
struct ScanPair {
  long long a;
  int b;
};
template <class Value, class Put>
__device__ ScanPair block_exclusive_scan2(int n, Value value, Put put, long long* scratch_a, int* scratch_b) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = (n + kPlanThreads - 1) / kPlanThreads;
  const int i0 = min(tid * chunk, n), i1 = min(i0 + chunk, n);
  ScanPair local = {0, 0};
  for (int i = i0; i < i1; ++i) {
    const ScanPair v = value(i);
    local.a += v.a;
    local.b += v.b;
  }
  ScanPair inc = local;
  for (int o = 1; o < 32; o <<= 1) {
    const long long xa = __shfl_up_sync(0xffffffffu, inc.a, o);
    const int xb = __shfl_up_sync(0xffffffffu, inc.b, o);
    if (lane >= o) {
      inc.a += xa;
      inc.b += xb;
    }
  }
  __syncthreads();                       // the scratch arrays may still be read by the previous scan
  if (lane == 31) {
    scratch_a[warp] = inc.a;
    scratch_b[warp] = inc.b;
  }
  __syncthreads();
  if (warp == 0) {
    const long long mine_a = scratch_a[lane];
    const int mine_b = scratch_b[lane];
    long long wa = mine_a;
    int wb = mine_b;
    for (int o = 1; o < 32; o <<= 1) {
      const long long xa = __shfl_up_sync(0xffffffffu, wa, o);
      const int xb = __shfl_up_sync(0xffffffffu, wb, o);
      if (lane >= o) {
        wa += xa;
        wb += xb;
      }
    }
    scratch_a[lane] = wa - mine_a;       // exclusive prefixes of the warp totals
    scratch_b[lane] = wb - mine_b;
    if (lane == 31) {                    // grand totals
      scratch_a[32] = wa;
      scratch_b[32] = wb;
    }
  }
  __syncthreads();
  const ScanPair total = {scratch_a[32], scratch_b[32]};
  ScanPair run = {scratch_a[warp] + inc.a - local.a, scratch_b[warp] + inc.b - local.b};
  for (int i = i0; i < i1; ++i) {
    const ScanPair v = value(i);   // read before put(): put may overwrite what value reads
    put(i, run.a, run.b);
    run.a += v.a;
    run.b += v.b;
  }
  __syncthreads();
  return total;
}

// Quotients on the work line.  Every operand is below W * teams; when that product fits 31 bits (the usual case) the
// 32-bit divide is used, which is several times cheaper than the emulated 64-bit one.
__device__ __forceinline__ long long qdiv(long long a, long long b, bool small) {
  return small ? static_cast<long long>(static_cast<unsigned>(a) / static_cast<unsigned>(b)) : a / b;
}
__device__ __forceinline__ long long ceil_div(long long a, long long b, bool small) { return qdiv(a + b - 1, b, small); }

// Ancestor-or-self masks of one tree by one warp: lane l holds nodes l and l + 32 (and is given their parent entries).  Every node starts with its own bit and a pointer to its
// parent; each round ORs in the mask of the node pointed to and jumps the pointer to that node's pointer, so six rounds
// cover any path of up to 64 nodes.  Returns false (to all lanes) on an invalid entry.  anc[i >= n] is not written.
__device__ inline bool build_masks_warp(int par_lo, int par_hi, int n, uint64_t* anc, uint8_t* depth, int lane) {
  uint64_t mask[2];
  int ptr[2];
  bool ok = true;
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int i = lane + 32 * k;
    mask[k] = 0ull;
    ptr[k] = -1;
    if (i < n) {
      const int pi = k == 0 ? par_lo : par_hi;   // parent of node lane / of node lane + 32, loaded by the caller
      if (pi < -1 || pi >= i) ok = false;
      else {
        mask[k] = 1ull << i;
        ptr[k] = pi;
      }
    }
  }
  if (!__all_sync(0xffffffffu, ok)) return false;
#pragma unroll
  for (int round = 0; round < 6; ++round) {
    uint64_t add[2];
    int next[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int t = ptr[k] >= 0 ? ptr[k] : 0;
      // the pointed-to node lives in lane t & 31, slot t >> 5: fetch both slots and pick
      const uint64_t m0 = __shfl_sync(0xffffffffu, mask[0], t & 31), m1 = __shfl_sync(0xffffffffu, mask[1], t & 31);
      const int p0 = __shfl_sync(0xffffffffu, ptr[0], t & 31), p1 = __shfl_sync(0xffffffffu, ptr[1], t & 31);
      add[k] = ptr[k] >= 0 ? ((t >> 5) ? m1 : m0) : 0ull;
      next[k] = ptr[k] >= 0 ? ((t >> 5) ? p1 : p0) : -1;
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      mask[k] |= add[k];
      ptr[k] = next[k];
    }
  }
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int i = lane + 32 * k;
    if (i < n) {
      anc[i] = mask[k];
      if (depth) depth[i] = static_cast<uint8_t>(__popcll(mask[k]));
    }
  }
  return true;
}

// A super-unit occupies [us, ue) on the work line: `ovh` positions of fixed cost, then one position per KV tile of
// its line.  Its interior cuts are the share boundaries floor(c * W / teams) with us + ovh + snap <= boundary <=
// ue - snap: a contiguous range of c.  Returns their number and the first such c.
__device__ __forceinline__ int unit_cuts(long long us, long long ue, long long W, int teams, int snap, int ovh, int* first_c, bool small) {
  const long long y = us + ovh + snap, z = ue - snap;
  *first_c = 0;
  if (z < y || teams < 2) return 0;
  long long ca = ceil_div(y * teams, W, small), cb = ceil_div((z + 1) * teams, W, small) - 1;
  if (ca < 1) ca = 1;
  if (cb > teams - 1) cb = teams - 1;
  *first_c = static_cast<int>(ca);
  return cb >= ca ? static_cast<int>(cb - ca + 1) : 0;
}

constexpr int kSmemSeqs = 512;     // per-sequence records kept in shared memory while planning (else in the workspace)
constexpr int kSmemUnits = 1792;   // per-super-unit records kept in shared memory while planning

// Geometry of a sequence's super-units.  The query tiles of one (sequence, KV head) are taken two at a time; such a
// PAIR is one super-unit whose line is the sequence's KV tiles (both CTAs of a team walk it, one query tile each).
// An odd last query tile has no sibling: the last tiles of two neighbouring KV heads form a TWIN super-unit with the
// same line (each CTA of the team walks it for its own head), and with an odd number of KV heads the last head's
// tile is a LONE super-unit whose line is half the KV tiles (the team's CTAs take one half each).  On the work line
// the heads are laid out two at a time: the pairs of head 2j, the pairs of head 2j + 1, their twin.
enum UnitKind { kPair = 0, kTwin = 1, kLone = 2 };
struct UnitGeom {
  int kind, g, mp, line;     // g: KV head (first of the two for a twin); mp: pair index within the head
  long long offset;          // start on the work line, relative to the sequence's start
};
struct SeqGeom {
  int pf, ntiles, half, plen, Hkv;   // whole pairs per head; KV tiles; ceil(ntiles/2); line + overhead of a pair or twin
  int u1, u2;                        // super-units of a leftover single head / of two heads
  long long len1, len2;              // line length of a leftover single head / of two heads
  bool odd;
  int ovh;
  __device__ SeqGeom(const SeqPlan& sp, int Hkv_, int ovh_) {
    Hkv = Hkv_;
    ovh = ovh_;
    pf = sp.mtiles / 2;
    ntiles = sp.ntiles;
    half = (sp.ntiles + 1) / 2;
    odd = (sp.mtiles & 1) != 0;
    plen = sp.ntiles + ovh;
    u1 = pf + (odd ? 1 : 0);
    u2 = 2 * pf + (odd ? 1 : 0);
    len1 = static_cast<long long>(pf) * plen + (odd ? half + ovh : 0);
    len2 = 2ll * pf * plen + (odd ? plen : 0);
  }
  __device__ int units() const { return (Hkv / 2) * u2 + (Hkv & 1) * u1; }
  __device__ long long length() const { return (Hkv / 2) * len2 + (Hkv & 1) * len1; }
  __device__ UnitGeom unit(int k) const {
    UnitGeom ug;
    const int twos = Hkv / 2;
    if (k < twos * u2) {
      const int h2 = k / u2, j = k % u2;
      const long long base = static_cast<long long>(h2) * len2;
      if (j < 2 * pf) {
        ug.kind = kPair;
        ug.g = 2 * h2 + (j >= pf ? 1 : 0);
        ug.mp = j >= pf ? j - pf : j;
        ug.offset = base + static_cast<long long>(j) * plen;
      } else {
        ug.kind = kTwin;
        ug.g = 2 * h2;
        ug.mp = pf;
        ug.offset = base + 2ll * pf * plen;
      }
      ug.line = ntiles;
    } else {
      const int j = k - twos * u2;
      const long long base = static_cast<long long>(twos) * len2;
      ug.g = Hkv - 1;
      ug.mp = j;
      ug.offset = base + static_cast<long long>(j) * plen;
      if (j < pf) {
        ug.kind = kPair;
        ug.line = ntiles;
      } else {
        ug.kind = kLone;
        ug.line = half;
      }
    }
    return ug;
  }
  // the super-unit that holds line position `off` (relative to the sequence's start, 0 <= off < length())
  __device__ int unit_at(long long off, bool small) const {
    const int twos = Hkv / 2;
    if (off < twos * len2) {
      const int h2 = static_cast<int>(qdiv(off, len2, small));
      int j = static_cast<int>(qdiv(off - h2 * len2, plen, small));
      if (j > u2 - 1) j = u2 - 1;
      return h2 * u2 + j;
    }
    int j = static_cast<int>(qdiv(off - twos * len2, plen, small));
    if (j > u1 - 1) j = u1 - 1;
    return twos * u2 + j;
  }
};

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(PlanParams pg) {
  __shared__ long long s_scan[kPlanThreads / 32 + 1];
  __shared__ int s_scan_b[kPlanThreads / 32 + 1];
  __shared__ int s_ncut;
  __shared__ SeqPlan s_seq[kSmemSeqs];
  __shared__ UnitPlan s_units[kSmemUnits];
  const int tid = threadIdx.x;
  if (tid == 0) s_ncut = 0;   // (the block synchronises several times before the counter is used)
  // The planning passes are chains of dependent reads and writes of these small tables; in shared memory each
  // link costs tens of cycles instead of a trip to L2.  They are copied to the workspace once at the end.
  PlanParams p = pg;
  const bool seq_in_smem = p.B <= kSmemSeqs, units_in_smem = p.unit_cap <= kSmemUnits;
  if (seq_in_smem) p.seq = s_seq;
  if (units_in_smem) p.units = s_units;
  const int T = p.T_max;
  const int ovh = p.forced_splits > 0 ? 0 : p.item_overhead_tiles;

  // ---- per sequence (one warp each): validate, build masks, count tiles.  The inputs of a warp's next sequence are
  // requested before the current one is worked on, and none of the loads depends on another's value.
  {
    const int lane = tid & 31;
    struct SeqIn {
      int n, L, par_lo, par_hi;
    };
    auto fetch = [&](int b) {
      SeqIn in;
      const int tb = p.shared_tree ? 0 : b;   // one tree for every sequence, or one per sequence
      const int32_t* par = p.tree_parent + static_cast<size_t>(tb) * T;
      in.n = p.tree_sizes ? p.tree_sizes[tb] : T;
      in.L = p.seq_lens[b];
      in.par_lo = lane < T ? par[lane] : -1;
      in.par_hi = lane + 32 < T ? par[lane + 32] : -1;
      return in;
    };
    int b = tid >> 5;
    SeqIn cur = {0, 0, -1, -1};
    if (b < p.B) cur = fetch(b);
    for (; b < p.B; b += kPlanThreads / 32) {
      SeqIn next = {0, 0, -1, -1};
      if (b + kPlanThreads / 32 < p.B) next = fetch(b + kPlanThreads / 32);
      int n = cur.n, L = cur.L;
      int bad = 0;
      if (n < 0 || n > T) bad = EAGLE_ERR_TREE;
      else if (L < 0 || static_cast<long long>(L) + n > p.S_cap) bad = EAGLE_ERR_SEQ;
      uint64_t* anc = p.anc + static_cast<size_t>(b) * T;
      if (!bad && !build_masks_warp(cur.par_lo, cur.par_hi, n, anc, nullptr, lane)) bad = EAGLE_ERR_TREE;
      if (!bad && p.block_table && n > 0) {
        // paged cache: every page that holds a visible slot must exist
        const int used = (L + n + p.page_size - 1) / p.page_size;
        bool page_ok = true;
        for (int i = lane; i < used; i += 32) {
          const int page = p.block_table[static_cast<size_t>(b) * p.max_pages + i];
          if (page < 0 || page >= p.num_pages) page_ok = false;
        }
        if (!__all_sync(0xffffffffu, page_ok)) bad = EAGLE_ERR_PAGE;
      }
      if (bad) {
        if (lane == 0) report_status(p.status, bad);
        n = 0;
        L = 0;
      }
      for (int i = n + lane; i < T; i += 32) anc[i] = 0ull;
      if (lane == 0) {
        SeqPlan sp;
        sp.n = n;
        sp.L = L;
        sp.mtiles = (n * p.G + kBlockM - 1) / kBlockM;
        sp.ntiles = n > 0 ? (L + n + p.tile_keys - 1) / p.tile_keys : 0;
        sp.unit_base = 0;
        sp.pad0 = 0;
        sp.start = 0;
        p.seq[b] = sp;
      }
      cur = next;
    }
  }
  __syncthreads();

  // ---- lay the sequences' super-units end to end
  const ScanPair WU = block_exclusive_scan2(
      p.B,
      [&](int b) {
        const SeqGeom ge(p.seq[b], p.Hkv, ovh);
        return ScanPair{ge.length(), ge.units()};
      },
      [&](int b, long long start, int unit_base) {
        p.seq[b].start = start;
        p.seq[b].unit_base = unit_base;
      },
      s_scan, s_scan_b);
  const long long W = WU.a, U = WU.b;
  const int n_units = U <= p.unit_cap ? static_cast<int>(U) : 0;   // cannot exceed the advertised workspace
  if (U > p.unit_cap && tid == 0) report_status(p.status, EAGLE_ERR_WORKSPACE);
  const int max_teams = p.num_ctas / 2;
  const int teams = static_cast<int>(W < max_teams ? (W > 0 ? W : 1) : max_teams);   // a share is at least one position
  const int snap = p.snap_tiles;
  const bool small = (W + ovh + snap + 1) * static_cast<long long>(max_teams + 1) < (1ll << 31);   // every dividend fits 31 bits

  // super-unit -> sequence: the last sequence whose unit_base <= u (sequences without units share theirs with the next)
  auto unit_seq = [&](int u) {
    int lo = 0, hi = p.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (p.seq[mid].unit_base <= u) lo = mid; else hi = mid;
    }
    return lo;
  };

  // ---- team pieces per super-unit
  for (int u = tid; u < n_units; u += kPlanThreads) {
    const int b = unit_seq(u);
    const SeqPlan sp = p.seq[b];
    const SeqGeom ge(sp, p.Hkv, ovh);
    const UnitGeom ug = ge.unit(u - sp.unit_base);
    const int len = ug.line;
    const long long us = sp.start + ug.offset;
    int np;
    if (p.forced_splits > 0) {
      np = len < p.forced_splits ? len : p.forced_splits;
    } else {
      int c0;
      np = 1 + unit_cuts(us, us + len + ovh, W, teams, snap, ovh, &c0, small);
    }
    p.units[u].n_pieces = np;
    p.units[u].pad0 = b;
  }
  __syncthreads();
  // a super-unit needs partial slots when some query tile of it ends up in more than one item:
  // a pair cut into np > 1 team pieces (np items per tile), or a single tile (its halves: 2 * np items) with > 1 KV tile
  auto slots_of = [&](int u) -> long long {
    const UnitPlan up = p.units[u];
    const SeqPlan sp = p.seq[up.pad0];
    const SeqGeom ge(sp, p.Hkv, ovh);
    const bool partial = ge.unit(u - sp.unit_base).kind != kLone ? up.n_pieces > 1 : sp.ntiles > 1;
    return partial ? 2ll * up.n_pieces : 0ll;
  };
  const ScanPair TS = block_exclusive_scan2(
      n_units, [&](int u) { return ScanPair{static_cast<long long>(p.units[u].n_pieces), static_cast<int>(slots_of(u))}; },
      [&](int u, long long first_item, int slot_base) {
        const bool has_slots = slots_of(u) > 0;     // (read before first_item is written: slots_of does not read it)
        p.units[u].first_item = static_cast<int>(first_item);
        p.units[u].slot_base = has_slots ? slot_base : -1;
      },
      s_scan, s_scan_b);
  const long long TP = TS.a, S = TS.b;
  const bool fits = 2 * TP <= p.item_cap && S <= p.slot_cap;
  if (!fits && tid == 0) report_status(p.status, EAGLE_ERR_WORKSPACE);   // cannot happen with the advertised size

  // ---- items: two per team piece, one for each CTA of the team.  The last warps do not take part: they fill the
  // teams' table and copy the tables out meanwhile (neither needs the items).
  constexpr int kSideThreads = 160, kMainThreads = kPlanThreads - kSideThreads;
  if (fits && tid < kMainThreads) {
    for (int u = tid; u < n_units; u += kMainThreads) {
      const UnitPlan up = p.units[u];
      const int b = up.pad0;
      const SeqPlan sp = p.seq[b];
      const SeqGeom ge(sp, p.Hkv, ovh);
      const UnitGeom ug = ge.unit(u - sp.unit_base);
      const int g = ug.g, mp = ug.mp;
      const bool paired = ug.kind != kLone;         // both CTAs of the team walk the same KV range
      const int len = ug.line, rest = sp.ntiles - len;      // lone tile: the second CTA's part has `rest` tiles
      const long long us = sp.start + ug.offset;
      const long long t_origin = us + ovh;          // line position of the super-unit's tile position 0
      int c0 = 0;
      if (p.forced_splits == 0) unit_cuts(us, us + len + ovh, W, teams, snap, ovh, &c0, small);
      bool live0 = false, live1 = false;    // query tiles of the super-unit with at least one non-empty item
      for (int j = 0; j < up.n_pieces; ++j) {
        int t0, t1;
        if (p.forced_splits > 0) {
          t0 = static_cast<int>(static_cast<long long>(len) * j / up.n_pieces);
          t1 = static_cast<int>(static_cast<long long>(len) * (j + 1) / up.n_pieces);
        } else {
          t0 = j == 0 ? 0 : static_cast<int>(qdiv(static_cast<long long>(c0 + j - 1) * W, teams, small) - t_origin);
          t1 = j == up.n_pieces - 1 ? len : static_cast<int>(qdiv(static_cast<long long>(c0 + j) * W, teams, small) - t_origin);
        }
        for (int m = 0; m < 2; ++m) {
          WorkItem it;
          it.b = b;
          it.g = ug.kind == kTwin ? g + m : g;
          if (paired) {
            it.mt = ug.kind == kTwin ? 2 * mp : 2 * mp + m;
            it.tile_begin = t0;
            it.tile_end = t1;
            it.slot = up.slot_base >= 0 ? up.slot_base + m * up.n_pieces + j : -1;
          } else {
            it.mt = 2 * mp;
            it.tile_begin = m == 0 ? t0 : len + (t0 < rest ? t0 : rest);
            it.tile_end = m == 0 ? t1 : len + (t1 < rest ? t1 : rest);
            it.slot = up.slot_base >= 0 ? up.slot_base + 2 * j + m : -1;
          }
          it.pad0 = it.pad1 = 0;
          p.items[2 * (up.first_item + j) + m] = it;
          if (it.tile_end > it.tile_begin) {
            if (paired && m == 1) live1 = true; else live0 = true;
          }
        }
      }
      // the query tiles whose pieces the combine kernel has to merge: a tile of a pair or twin is spread over one
      // member's items (every second item), a lone tile over the items of both CTAs
      if (up.slot_base >= 0) {
        for (int m = 0; m < 2; ++m) {
          if (!(m == 0 ? live0 : live1)) continue;
          CutTile ct;
          ct.b = b;
          ct.g = ug.kind == kTwin ? g + m : g;
          ct.mt = ug.kind == kPair ? 2 * mp + m : 2 * mp;
          ct.m_valid = sp.n * p.G;
          ct.item0 = 2 * up.first_item + (paired ? m : 0);
          ct.item_stride = paired ? 2 : 1;
          ct.slot0 = up.slot_base + (paired ? m * up.n_pieces : 0);
          ct.count = paired ? up.n_pieces : 2 * up.n_pieces;
          pg.cut_tiles[atomicAdd(&s_ncut, 1)] = ct;
        }
      }
    }
  }

  // ---- first team piece of every team (cta_first is indexed by team here; entries past the last team repeat the end)
  for (int c = tid - kMainThreads; c >= 0 && c <= p.num_ctas; c += kSideThreads) {
    long long first;
    if (!fits || TP == 0) {
      first = 0;
    } else if (p.forced_splits > 0) {
      first = c >= max_teams ? TP : static_cast<long long>(c) * TP / max_teams;
    } else if (c == 0) {
      first = 0;
    } else if (c >= teams) {
      first = TP;
    } else {
      const long long x = qdiv(static_cast<long long>(c) * W, teams, small);   // 0 < x < W
      int lo = 0, hi = p.B;          // last sequence whose start <= x (sequences without work share their start with the next)
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.seq[mid].start <= x) lo = mid; else hi = mid;
      }
      const SeqPlan sp = p.seq[lo];
      const SeqGeom ge(sp, p.Hkv, ovh);
      const int k = ge.unit_at(x - sp.start, small);
      const UnitGeom ug = ge.unit(k);
      const int u = sp.unit_base + k;
      const long long us = sp.start + ug.offset, ue = us + ug.line + ovh;
      const long long d0 = x - (us + ovh), d1 = ue - x;   // distance to the first tile position / to the super-unit's end
      const UnitPlan up = p.units[u];
      if (d0 >= snap && d1 >= snap) {
        int c0;
        unit_cuts(us, ue, W, teams, snap, ovh, &c0, small);
        first = up.first_item + 1 + (c - c0);        // the piece that starts at this boundary
      } else if (x - us <= d1) {
        first = up.first_item;                        // boundary moved to the super-unit's start
      } else {
        first = up.first_item + up.n_pieces;          // boundary moved to the super-unit's end
      }
    }
    p.cta_first[c] = static_cast<int>(first);
  }
  if (tid >= kMainThreads) {
    if (seq_in_smem)
      for (int b = tid - kMainThreads; b < p.B; b += kSideThreads) pg.seq[b] = s_seq[b];
    if (units_in_smem)
      for (int u = tid - kMainThreads; u < n_units; u += kSideThreads) pg.units[u] = s_units[u];
  }
  __syncthreads();
  if (tid == 0) {
    p.hdr->n_items = fits ? static_cast<int>(2 * TP) : 0;
    p.hdr->n_slots = fits ? static_cast<int>(S) : 0;
    p.hdr->n_units = n_units;
    p.hdr->n_cut = s_ncut;
    p.hdr->ctas_used = 2 * teams;
    p.hdr->total_tiles = W;
  }
}

// The stand-alone mask builder: one warp per tree, the same routine the planner runs.
constexpr int kMaskWarps = 4;
__global__ void __launch_bounds__(32 * kMaskWarps)
build_mask_kernel(const int32_t* __restrict__ tree_parent, const int32_t* __restrict__ tree_sizes, int batch, int T,
                  uint64_t* __restrict__ anc, uint8_t* __restrict__ depth, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * kMaskWarps + (threadIdx.x >> 5);
  if (b >= batch) return;   // uniform over the warp
  int n = tree_sizes ? tree_sizes[b] : T;
  const int32_t* par = tree_parent + static_cast<size_t>(b) * T;
  uint64_t* a = anc + static_cast<size_t>(b) * T;
  uint8_t* d = depth ? depth + static_cast<size_t>(b) * T : nullptr;
  bool ok = n >= 0 && n <= T;
  if (ok) ok = build_masks_warp(lane < n ? par[lane] : -1, lane + 32 < n ? par[lane + 32] : -1, n, a, d, lane);
  if (!ok) {
    if (lane == 0) report_status(status, EAGLE_ERR_TREE);
    n = 0;
  }
  for (int i = n + lane; i < T; i += 32) {
    a[i] = 0ull;
    if (d) d[i] = 0;
  }
}

}  // namespace

cudaError_t launch_plan(const PlanParams& p, cudaStream_t stream) {
  plan_kernel<<<1, kPlanThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int batch, int max_tree,
                              uint64_t* anc, uint8_t* depth, int32_t* status, cudaStream_t stream) {
  build_mask_kernel<<<(batch + kMaskWarps - 1) / kMaskWarps, 32 * kMaskWarps, 0, stream>>>(tree_parent, tree_sizes, batch, max_tree,
                                                                                            anc, depth, status);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
