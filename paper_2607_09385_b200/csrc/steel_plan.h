// Plain-data structures shared by the host planner and the device kernel: work items, step
// entries and kernel parameters.  The planner turns the mask descriptor into these (the three
// mask cases of the paper's Sec. "The STEEL Pipeline" at 128 x 128 tile granularity); the kernel
// only ever sees tiles that must be executed.
#pragma once
#include <stdint.h>

namespace steel {

constexpr int kTile = 128;  // query rows per tile and keys per tile
constexpr long long kDefaultTimeoutCycles = 4000000000ll;  // about two seconds of SM clock

// One step entry of one query tile ("slot") in a list-kind item.
constexpr uint32_t kEntryTileMask = 0x00FFFFFFu;  // key-tile index
constexpr uint32_t kEntryPresent = 1u << 24;
constexpr uint32_t kEntryPartial = 1u << 25;      // element-wise mask needed
constexpr uint32_t kEntrySubShift = 26;           // 4 bits: 64x64 sub-blocks TL, TR, BL, BR enabled
constexpr uint32_t kEntrySubAll = 0xFu << kEntrySubShift;

// A work item: one or two query tiles ("slots") of the same batch and KV head that walk their key
// tiles in lock-step, sharing a K/V load whenever both want the same key tile at the same step.
// Slot s is present on steps lo[s]..hi[s] (inclusive; lo > hi means the slot is unused), and
// lo[0] <= lo[1] whenever both are used.
struct WorkItem {
  int32_t batch;
  int32_t kv_head;
  int32_t head[2];   // query head of each slot
  int32_t qtile[2];  // query tile index (rows qtile*128 ...) of each slot
  int32_t lo[2];
  int32_t hi[2];
  int32_t n_steps;
  int32_t kind;      // 0: range (key tile of step t is j0 + t for both slots), 1: list
  int32_t j0;        // range kind
  int32_t list_off;  // list kind: index of the item's first StepPair
  int32_t cost;      // executed tiles
  int32_t pad;
};
static_assert(sizeof(WorkItem) == 64, "WorkItem layout");

// Entries of both slots for one step of a list-kind item.
struct StepPair {
  uint32_t e[2];
};

struct KernelParams {
  const WorkItem *items;     // ordered so that CTA c owns items cta_begin[c] .. cta_begin[c+1]-1
  const int32_t *cta_begin;  // gridDim.x + 1 entries
  const StepPair *steps;       // list-kind step entries
  void *o;                   // bf16 [batch, heads_q, seq_q, head_dim]
  float *lse;                // fp32 [batch, heads_q, seq_q] or null
  int32_t *status;           // device status word (0 ok, else STEEL_ERR_TIMEOUT)
  int32_t heads_q, heads_kv, seq_q, seq_kv;
  uint32_t mask_flags;
  int32_t window;            // clamped to int32 range
  float scale_log2;          // scale * log2(e)
  long long *trace;          // per-CTA wait accounting (debug builds only), else null
  long long *clock_probe;    // measurement hook: CTA 0 stores {SM cycles, nanoseconds} of its run here, else null
  long long timeout_cycles;  // bound of every device-side wait
  int32_t stall_cta;         // test hook: this CTA's producer withholds its commands (-1: none)
};

}  // namespace steel
