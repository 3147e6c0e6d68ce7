// Host planner interface: turns a validated problem description into the work items, step lists
// and per-CTA assignment the kernel consumes, and the statistics reported to callers.
#pragma once
#include <functional>
#include <vector>

#include "../../include/steel_attn.h"
#include "steel_plan.h"

namespace steel {

// K + V bytes of the KV heads scheduled together.  Data that every SM reads ends up in both halves
// of the 126 MB L2, so about half of it is usable: with 64 MiB waves the 32K bitmap workload read its
// K/V from DRAM 1.5 times, with 32 MiB waves 1.02 times (and ran 2 % faster).
constexpr int64_t kL2WaveBytes = 32ll << 20;
// Fixed cost of an item (Q load, first-tile latency, epilogue) in units of one key-tile step.
constexpr int kItemOverheadSteps = 2;
// Bitmap masks: how many tasks of similar length are examined when choosing a query tile's partner.
constexpr size_t kPartnerWindow = 16;
// CTA count assumed by the host-only planning entry point (the SM count of a B200).
constexpr int kPlanHostCtas = 148;

struct Plan {
  std::vector<WorkItem> items;     // in CTA order
  std::vector<int32_t> cta_begin;  // grid + 1
  std::vector<StepPair> steps;     // list-kind entries
  steel_attn_stats_t stats;
  int grid = 0;
};

steel_status_t validate_params(const steel_attn_params_t *p);
// Scheduling policy and the other options come from `p`.  `exec_stats` = false skips the statistics
// that need a walk over every executed tile (exec_tiles, exec_partial, kv_tile_loads stay 0).
steel_status_t build_plan(const steel_attn_params_t *p, int num_ctas, Plan *plan, bool exec_stats = true);

// Entry (tile index and flags, 0 if absent) of `slot` at step `t`, derived exactly as on the device.
uint32_t item_entry(const Plan &plan, const WorkItem &w, int slot, int t, const steel_attn_params_t *p);

// Visit every executed tile: (item index, item, slot, step, entry, shares the other slot's load).
void walk_plan(const Plan &plan, const std::function<void(int, const WorkItem &, int, int, uint32_t, bool)> &visit,
               const steel_attn_params_t *p);

}  // namespace steel
