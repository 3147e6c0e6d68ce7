// Host planner: mask descriptor -> executed-tile lists -> work items -> per-CTA assignment.
// Pure host C++ (no CUDA calls), so it is testable on a machine without a GPU.
#include "steel_planner.h"

#include <algorithm>
#include <cmath>
#include <limits>
#include <queue>

namespace steel {
namespace {

constexpr int64_t kInf = std::numeric_limits<int64_t>::max() / 4;

// Geometry of the causal / window terms of the predicate, on token rectangles with inclusive
// bounds that lie inside the problem.  `p = i + off` is the key position aligned with query i.
struct Geom {
  int64_t seq_q, seq_kv, off, window;
  bool causal, windowed;

  bool any_visible(int64_t i0, int64_t i1, int64_t j0, int64_t j1) const {
    // row p sees keys (p - W, p]; it meets [j0, j1] iff j0 <= p (causal) and p <= j1 + W - 1 (window)
    int64_t lb = causal ? j0 : -kInf, ub = windowed ? j1 + window - 1 : kInf;
    return std::max(lb, i0 + off) <= std::min(ub, i1 + off);
  }
  bool all_visible(int64_t i0, int64_t i1, int64_t j0, int64_t j1) const {
    if (causal && !(j1 <= i0 + off)) return false;
    if (windowed && !((i1 + off) - j0 < window)) return false;
    return true;
  }
  int64_t visible_pairs(int64_t i0, int64_t i1, int64_t j0, int64_t j1) const {
    if (all_visible(i0, i1, j0, j1)) return (i1 - i0 + 1) * (j1 - j0 + 1);
    int64_t n = 0;
    for (int64_t i = i0; i <= i1; ++i) {
      int64_t p = i + off;
      int64_t a = std::max(j0, windowed ? p - window + 1 : -kInf), b = std::min(j1, causal ? p : kInf);
      if (b >= a) n += b - a + 1;
    }
    return n;
  }
};

struct Ctx {
  const steel_attn_params_t *p;
  Geom g;
  int64_t bq, bkv;         // descriptor block sizes (64 or 128)
  int64_t tq128, tkv128;   // kernel tiles
  int64_t tqb, tkvb, words;  // descriptor blocks
  bool bitmap;

  bool bit(int h, int64_t I, int64_t J) const {
    if (I >= tqb || J >= tkvb) return false;
    return (p->mask.bitmap[(int64_t(h) * tqb + I) * words + (J >> 5)] >> (J & 31)) & 1u;
  }
  void rows(int64_t I, int64_t size, int64_t &i0, int64_t &i1) const {
    i0 = I * size;
    i1 = std::min<int64_t>(i0 + size - 1, p->seq_q - 1);
  }
  void keys(int64_t J, int64_t size, int64_t &j0, int64_t &j1) const {
    j0 = J * size;
    j1 = std::min<int64_t>(j0 + size - 1, p->seq_kv - 1);
  }
  // Entry of kernel tile (I, J) for head h, or 0 if the tile is fully masked (case i).
  uint32_t entry(int h, int64_t I, int64_t J) const {
    int64_t i0, i1, j0, j1;
    rows(I, kTile, i0, i1);
    keys(J, kTile, j0, j1);
    bool ragged = (j1 - j0 + 1) < kTile;
    uint32_t sub = 0xF;
    bool kept, full;
    if (!bitmap) {
      kept = g.any_visible(i0, i1, j0, j1);
      full = g.all_visible(i0, i1, j0, j1);
    } else if (bq == kTile) {
      kept = bit(h, I, J) && g.any_visible(i0, i1, j0, j1);
      full = g.all_visible(i0, i1, j0, j1);
    } else {  // 64-token blocks: four sub-blocks TL, TR, BL, BR
      sub = 0;
      kept = false;
      full = g.all_visible(i0, i1, j0, j1);
      for (int a = 0; a < 2; ++a)
        for (int b = 0; b < 2; ++b) {
          int64_t si0 = i0 + 64 * a, sj0 = j0 + 64 * b;
          if (si0 > i1 || sj0 > j1) continue;  // outside the problem
          int64_t si1 = std::min(si0 + 63, i1), sj1 = std::min(sj0 + 63, j1);
          if (bit(h, 2 * I + a, 2 * J + b)) {
            sub |= 1u << (2 * a + b);
            kept = kept || g.any_visible(si0, si1, sj0, sj1);
          } else {
            full = false;
          }
        }
    }
    if (!kept) return 0;
    uint32_t e = uint32_t(J) | kEntryPresent | (sub << kEntrySubShift);
    if (!full || ragged) e |= kEntryPartial;
    return e;
  }
};

struct Task {  // one query tile of one head
  int h;
  int64_t I;
  int64_t jlo = 0, jhi = -1;      // range kind
  std::vector<uint32_t> entries;  // list kind
  int64_t count() const { return entries.empty() ? jhi - jlo + 1 : int64_t(entries.size()); }
};

}  // namespace

steel_status_t validate_params(const steel_attn_params_t *p) {
  if (!p) return STEEL_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->seq_q <= 0 || p->seq_kv <= 0 || p->head_dim <= 0)
    return STEEL_ERR_INVALID_ARG;
  if (p->heads_q % p->heads_kv != 0) return STEEL_ERR_INVALID_ARG;
  if (!(p->scale > 0.0f) || !std::isfinite(p->scale)) return STEEL_ERR_INVALID_ARG;
  const uint32_t known = STEEL_MASK_CAUSAL | STEEL_MASK_WINDOW | STEEL_MASK_BITMAP;
  if (p->mask.flags & ~known) return STEEL_ERR_INVALID_ARG;
  if ((p->mask.flags & STEEL_MASK_WINDOW) && p->mask.window <= 0) return STEEL_ERR_INVALID_ARG;
  if ((p->mask.flags & STEEL_MASK_BITMAP) && !p->mask.bitmap) return STEEL_ERR_INVALID_ARG;
  if (p->mask.block_q < 0 || p->mask.block_kv < 0) return STEEL_ERR_INVALID_ARG;
  if (p->policy < 0 || p->policy > 2 || p->exp_emulation < 0 || p->exp_emulation > 3) return STEEL_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return STEEL_ERR_UNSUPPORTED;
  int bq = p->mask.block_q ? p->mask.block_q : kTile, bkv = p->mask.block_kv ? p->mask.block_kv : kTile;
  if (bq != bkv || (bq != 64 && bq != 128)) return STEEL_ERR_UNSUPPORTED;
  if ((int64_t(p->seq_kv) + kTile - 1) / kTile > (int64_t(1) << 24)) return STEEL_ERR_UNSUPPORTED;
  if (p->seq_q > (1 << 30) || p->seq_kv > (1 << 30)) return STEEL_ERR_UNSUPPORTED;
  if (int64_t(p->batch) * p->heads_q * p->seq_q >= (int64_t(1) << 31)) return STEEL_ERR_UNSUPPORTED;
  if (int64_t(p->batch) * p->heads_kv * p->seq_kv >= (int64_t(1) << 31)) return STEEL_ERR_UNSUPPORTED;
  return STEEL_OK;
}

steel_status_t build_plan(const steel_attn_params_t *p, int num_ctas, Plan *plan, bool exec_stats) {
  steel_status_t st = validate_params(p);
  if (st != STEEL_OK) return st;
  const int policy = p->policy;
  if (num_ctas <= 0 || !plan) return STEEL_ERR_INVALID_ARG;

  Ctx c;
  c.p = p;
  c.bitmap = (p->mask.flags & STEEL_MASK_BITMAP) != 0;
  c.g = Geom{p->seq_q, p->seq_kv, int64_t(p->seq_kv) - p->seq_q, p->mask.window,
             (p->mask.flags & STEEL_MASK_CAUSAL) != 0, (p->mask.flags & STEEL_MASK_WINDOW) != 0};
  c.bq = p->mask.block_q ? p->mask.block_q : kTile;
  c.bkv = p->mask.block_kv ? p->mask.block_kv : kTile;
  c.tq128 = (p->seq_q + kTile - 1) / kTile;
  c.tkv128 = (p->seq_kv + kTile - 1) / kTile;
  c.tqb = (p->seq_q + c.bq - 1) / c.bq;
  c.tkvb = (p->seq_kv + c.bkv - 1) / c.bkv;
  c.words = (c.tkvb + 31) / 32;
  const int G = p->heads_q / p->heads_kv;

  plan->items.clear();
  plan->steps.clear();
  plan->cta_begin.clear();
  steel_attn_stats_t &s = plan->stats;
  s = steel_attn_stats_t{};

  // ---- statistics at the descriptor's block granularity (what "kept tiles" means to a caller)
  {
    int64_t kept = 0, partial = 0;
    double pairs = 0.0;
    for (int h = 0; h < p->heads_q; ++h) {
      if (!c.bitmap && h > 0) break;  // range masks are identical for every head
      for (int64_t I = 0; I < c.tqb; ++I) {
        int64_t i0, i1;
        c.rows(I, c.bq, i0, i1);
        for (int64_t J = 0; J < c.tkvb; ++J) {
          if (c.bitmap && !c.bit(h, I, J)) continue;
          int64_t j0, j1;
          c.keys(J, c.bkv, j0, j1);
          if (!c.g.any_visible(i0, i1, j0, j1)) {
            if (!c.bitmap && c.g.causal && j0 > i1 + c.g.off) break;  // rest of the row is empty
            continue;
          }
          ++kept;
          bool full = c.g.all_visible(i0, i1, j0, j1);
          partial += !full;
          pairs += full ? double((i1 - i0 + 1) * (j1 - j0 + 1)) : double(c.g.visible_pairs(i0, i1, j0, j1));
        }
      }
    }
    int64_t mult = int64_t(p->batch) * (c.bitmap ? 1 : p->heads_q);
    s.kept_tiles = kept * mult;
    s.partial_tiles = partial * mult;
    s.total_tiles = int64_t(p->batch) * p->heads_q * c.tqb * c.tkvb;
    s.effective_flop = 4.0 * double(c.bq) * double(c.bkv) * p->head_dim * double(s.kept_tiles);
    s.useful_flop = 4.0 * p->head_dim * pairs * double(mult);
  }

  // ---- per (head, query tile) executed key tiles
  std::vector<std::vector<Task>> tasks(p->heads_q);  // [h][I]
  for (int h = 0; h < p->heads_q; ++h) {
    tasks[h].resize(c.tq128);
    for (int64_t I = 0; I < c.tq128; ++I) {
      Task &t = tasks[h][I];
      t.h = h;
      t.I = I;
      if (c.bitmap) {
        for (int64_t J = 0; J < c.tkv128; ++J) {
          uint32_t e = c.entry(h, I, J);
          if (e) t.entries.push_back(e);
        }
      } else if (h > 0) {
        t.jlo = tasks[0][I].jlo;
        t.jhi = tasks[0][I].jhi;
      } else {
        // kept key tiles of a row of tiles form one contiguous range under causal / window masks
        int64_t i0, i1;
        c.rows(I, kTile, i0, i1);
        int64_t p0 = i0 + c.g.off, p1 = i1 + c.g.off;
        int64_t hi = c.g.causal ? std::min<int64_t>(c.tkv128 - 1, p1 >= 0 ? p1 / kTile : -1) : c.tkv128 - 1;
        int64_t lo = 0;
        if (c.g.windowed) {
          int64_t first_key = p0 - c.g.window + 1;
          lo = first_key > 0 ? first_key / kTile : 0;
        }
        while (lo <= hi && !c.entry(0, I, lo)) ++lo;
        while (hi >= lo && !c.entry(0, I, hi)) --hi;
        t.jlo = lo;
        t.jhi = hi;
      }
    }
  }

  // ---- work items: pair query tiles that can share K/V loads
  struct Draft {
    WorkItem w;
    std::vector<StepPair> list;
    int group;
  };
  std::vector<Draft> drafts;
  auto finish_range = [&](const Task *a, const Task *b, int batch, int g) {
    Draft d{};
    d.group = g;
    WorkItem &w = d.w;
    w.batch = batch;
    w.kv_head = g;
    w.kind = 0;
    w.head[0] = a->h;
    w.qtile[0] = int32_t(a->I);
    w.head[1] = b ? b->h : -1;
    w.qtile[1] = b ? int32_t(b->I) : 0;
    w.j0 = int32_t(a->jlo);
    w.lo[0] = 0;
    w.hi[0] = int32_t(a->jhi - a->jlo);
    w.lo[1] = 1;
    w.hi[1] = 0;
    if (b) {
      w.lo[1] = int32_t(b->jlo - a->jlo);
      w.hi[1] = int32_t(b->jhi - a->jlo);
    }
    w.n_steps = std::max(w.hi[0], w.hi[1]) + 1;
    w.cost = int32_t(a->count() + (b ? b->count() : 0));
    drafts.push_back(std::move(d));
  };
  auto finish_list = [&](const Task *a, const Task *b, int batch, int g) {
    Draft d{};
    d.group = g;
    WorkItem &w = d.w;
    w.batch = batch;
    w.kv_head = g;
    w.kind = 1;
    w.head[0] = a->h;
    w.qtile[0] = int32_t(a->I);
    w.head[1] = b ? b->h : -1;
    w.qtile[1] = b ? int32_t(b->I) : 0;
    size_t na = a->entries.size(), nb = b ? b->entries.size() : 0;
    w.lo[0] = 0;
    w.hi[0] = int32_t(na) - 1;
    w.lo[1] = b ? 0 : 1;
    w.hi[1] = b ? int32_t(nb) - 1 : 0;
    w.n_steps = int32_t(std::max(na, nb));
    // Key tiles may be visited in any order (the online softmax does not care), so the tiles both
    // query tiles want come first, in the same steps: each of those steps needs one K/V load, not two.
    std::vector<uint32_t> ea, eb;
    if (b) {
      std::vector<uint32_t> rest_a, rest_b;
      size_t ia = 0, ib = 0;
      while (ia < na || ib < nb) {
        const uint32_t ta = ia < na ? (a->entries[ia] & kEntryTileMask) : 0xFFFFFFFFu;
        const uint32_t tb = ib < nb ? (b->entries[ib] & kEntryTileMask) : 0xFFFFFFFFu;
        if (ta == tb) {
          ea.push_back(a->entries[ia++]);
          eb.push_back(b->entries[ib++]);
        } else if (ta < tb) {
          rest_a.push_back(a->entries[ia++]);
        } else {
          rest_b.push_back(b->entries[ib++]);
        }
      }
      ea.insert(ea.end(), rest_a.begin(), rest_a.end());
      eb.insert(eb.end(), rest_b.begin(), rest_b.end());
    } else {
      ea = a->entries;
    }
    for (size_t t = 0; t < size_t(w.n_steps); ++t)
      d.list.push_back(StepPair{{t < na ? ea[t] : 0u, t < nb ? eb[t] : 0u}});
    w.cost = int32_t(na + nb);
    drafts.push_back(std::move(d));
  };
  auto empty_item = [&](const Task *a, int batch, int g) {  // no visible key: rows get O = 0, LSE = -inf
    Draft d{};
    d.group = g;
    WorkItem &w = d.w;
    w.batch = batch;
    w.kv_head = g;
    w.kind = 0;
    w.head[0] = a->h;
    w.qtile[0] = int32_t(a->I);
    w.head[1] = -1;
    w.lo[0] = 0;
    w.hi[0] = -1;
    w.lo[1] = 1;
    w.hi[1] = 0;
    w.n_steps = 0;
    drafts.push_back(std::move(d));
  };

  for (int batch = 0; batch < p->batch; ++batch) {
    for (int g = 0; g < p->heads_kv; ++g) {
      std::vector<const Task *> live;
      for (int h = g * G; h < (g + 1) * G; ++h)
        for (int64_t I = 0; I < c.tq128; ++I) {
          const Task *t = &tasks[h][I];
          if (t->count() <= 0) empty_item(t, batch, g);
          else live.push_back(t);
        }
      if (c.bitmap) {
        // similar lengths pair best: both tiles of an item then finish together
        std::stable_sort(live.begin(), live.end(), [](const Task *a, const Task *b) { return a->count() > b->count(); });
        // among the next few tasks of similar length, take the partner with the most key tiles in common
        std::vector<bool> used(live.size(), false);
        for (size_t n = 0; n < live.size(); ++n) {
          if (used[n]) continue;
          used[n] = true;
          size_t best = live.size(), seen = 0;
          int64_t best_common = 0;
          for (size_t m = n + 1; m < live.size() && seen < kPartnerWindow; ++m) {
            if (used[m]) continue;
            ++seen;
            int64_t common = 0;
            size_t ia = 0, ib = 0;
            const std::vector<uint32_t> &ea = live[n]->entries, &eb = live[m]->entries;
            while (ia < ea.size() && ib < eb.size()) {
              const uint32_t ta = ea[ia] & kEntryTileMask, tb = eb[ib] & kEntryTileMask;
              if (ta == tb) { ++common; ++ia; ++ib; }
              else if (ta < tb) ++ia;
              else ++ib;
            }
            // a step with one idle slot costs far more than a shared load saves
            const int64_t score = common - 16 * (live[n]->count() - live[m]->count());
            if (score > best_common || best == live.size()) { best_common = score; best = m; }
          }
          if (best < live.size()) used[best] = true;
          finish_list(live[n], best < live.size() ? live[best] : nullptr, batch, g);
        }
      } else if (G % 2 == 0) {
        // two query heads of the group on the same query tile: identical key ranges
        for (int h = g * G; h < (g + 1) * G; h += 2)
          for (int64_t I = 0; I < c.tq128; ++I)
            if (tasks[h][I].count() > 0) finish_range(&tasks[h][I], &tasks[h + 1][I], batch, g);
      } else {
        // adjacent query tiles of one head: ranges differ by at most one tile at each end
        for (int h = g * G; h < (g + 1) * G; ++h) {
          int64_t I = 0;
          while (I < c.tq128) {
            const Task *a = &tasks[h][I];
            if (a->count() <= 0) { ++I; continue; }
            const Task *b = (I + 1 < c.tq128 && tasks[h][I + 1].count() > 0) ? &tasks[h][I + 1] : nullptr;
            if (b && (b->jlo < a->jlo || b->jlo > a->jhi + 1)) b = nullptr;
            finish_range(a, b, batch, g);
            I += b ? 2 : 1;
          }
        }
      }
    }
  }

  // ---- order: waves of KV heads whose K and V fit comfortably in L2, longest item first inside
  // a wave (policy 0); natural order (policy 1)
  std::vector<int> order(drafts.size());
  for (size_t n = 0; n < order.size(); ++n) order[n] = int(n);
  if (policy == 0) {
    const double kv_bytes_per_head = 2.0 * double(p->seq_kv) * p->head_dim * 2.0;
    int heads_per_wave = int(std::max(1.0, std::floor(double(kL2WaveBytes) / kv_bytes_per_head)));
    auto wave_of = [&](const Draft &d) { return (int64_t(d.w.batch) * p->heads_kv + d.group) / heads_per_wave; };
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      int64_t wa = wave_of(drafts[a]), wb = wave_of(drafts[b]);
      if (wa != wb) return wa < wb;
      return drafts[a].w.n_steps > drafts[b].w.n_steps;
    });
  }

  // ---- assignment to persistent CTAs
  int grid = int(std::min<size_t>(size_t(num_ctas), std::max<size_t>(drafts.size(), 1)));
  std::vector<std::vector<int>> per_cta(grid);
  std::vector<int64_t> load(grid, 0);
  if (policy == 0) {
    // greedy longest-processing-time: next item goes to the least loaded CTA
    typedef std::pair<int64_t, int> Slot;
    std::priority_queue<Slot, std::vector<Slot>, std::greater<Slot>> heap;
    for (int cta = 0; cta < grid; ++cta) heap.push(Slot(0, cta));
    for (int id : order) {
      Slot sl = heap.top();
      heap.pop();
      per_cta[sl.second].push_back(id);
      sl.first += drafts[id].w.n_steps + kItemOverheadSteps;
      load[sl.second] = sl.first;
      heap.push(sl);
    }
  } else if (policy == 1) {
    // uniform placement: contiguous chunks of the natural order
    size_t n = order.size();
    for (size_t k = 0; k < n; ++k) {
      int cta = int(k * size_t(grid) / std::max<size_t>(n, 1));
      per_cta[cta].push_back(order[k]);
      load[cta] += drafts[order[k]].w.n_steps + kItemOverheadSteps;
    }
  } else {
    // interleaved placement: consecutive items of the natural order go to consecutive CTAs, so
    // that CTAs working side by side hold query tiles of similar sparsity
    for (size_t k = 0; k < order.size(); ++k) {
      int cta = int(k % size_t(grid));
      per_cta[cta].push_back(order[k]);
      load[cta] += drafts[order[k]].w.n_steps + kItemOverheadSteps;
    }
  }

  plan->grid = grid;
  plan->cta_begin.push_back(0);
  for (int cta = 0; cta < grid; ++cta) {
    for (int id : per_cta[cta]) {
      Draft &d = drafts[id];
      if (d.w.kind == 1) {
        d.w.list_off = int32_t(plan->steps.size());
        plan->steps.insert(plan->steps.end(), d.list.begin(), d.list.end());
      }
      plan->items.push_back(d.w);
    }
    plan->cta_begin.push_back(int32_t(plan->items.size()));
  }
  if (plan->steps.size() >= (size_t(1) << 31)) return STEEL_ERR_UNSUPPORTED;

  // ---- statistics of the executed plan
  s.work_items = int64_t(plan->items.size());
  s.grid = grid;
  s.list_entries = int64_t(plan->steps.size());
  s.max_cta_steps = 0;
  for (int cta = 0; cta < grid; ++cta) {
    int64_t st_sum = 0;
    for (int id : per_cta[cta]) st_sum += drafts[id].w.n_steps;
    s.max_cta_steps = std::max(s.max_cta_steps, st_sum);
  }
  // the walk visits every executed tile (millions on long sequences): only for callers that read these
  if (exec_stats) walk_plan(*plan, [&](int, const WorkItem &, int, int, uint32_t entry, bool shared) {
    ++s.exec_tiles;
    s.exec_partial += (entry & kEntryPartial) != 0;
    s.kv_tile_loads += shared ? 0 : 1;
  }, p);
  for (const WorkItem &w : plan->items) s.steps += w.n_steps;
  return STEEL_OK;
}

// Entry of slot `slot` at step t of an item, as the kernel derives it.
uint32_t item_entry(const Plan &plan, const WorkItem &w, int slot, int t, const steel_attn_params_t *p) {
  if (w.head[slot] < 0 || t < w.lo[slot] || t > w.hi[slot]) return 0;
  if (w.kind == 1) return plan.steps[size_t(w.list_off) + size_t(t)].e[slot];
  // range kind: geometry decides whether the element-wise mask is needed
  Geom g{p->seq_q, p->seq_kv, int64_t(p->seq_kv) - p->seq_q, p->mask.window,
         (p->mask.flags & STEEL_MASK_CAUSAL) != 0, (p->mask.flags & STEEL_MASK_WINDOW) != 0};
  int64_t J = int64_t(w.j0) + t;
  int64_t i0 = int64_t(w.qtile[slot]) * kTile, i1 = std::min<int64_t>(i0 + kTile - 1, p->seq_q - 1);
  int64_t j0 = J * kTile, j1 = std::min<int64_t>(j0 + kTile - 1, p->seq_kv - 1);
  uint32_t e = uint32_t(J) | kEntryPresent | kEntrySubAll;
  if (!g.all_visible(i0, i1, j0, j1) || (j1 - j0 + 1) < kTile) e |= kEntryPartial;
  return e;
}

void walk_plan(const Plan &plan, const std::function<void(int, const WorkItem &, int, int, uint32_t, bool)> &visit,
               const steel_attn_params_t *p) {
  for (size_t n = 0; n < plan.items.size(); ++n) {
    const WorkItem &w = plan.items[n];
    for (int t = 0; t < w.n_steps; ++t) {
      uint32_t e0 = item_entry(plan, w, 0, t, p), e1 = item_entry(plan, w, 1, t, p);
      bool shared = e0 && e1 && ((e0 & kEntryTileMask) == (e1 & kEntryTileMask));
      if (e0) visit(int(n), w, 0, t, e0, false);
      if (e1) visit(int(n), w, 1, t, e1, shared);
    }
  }
}

}  // namespace steel
