// Fused block-sparse attention kernel for sm_100a (paper Algorithm 1 on one persistent CTA per SM).
//
// A CTA processes work items; an item is one or two query tiles (128 rows each, "slots") that walk
// the same sequence of key-tile steps.  Roles (three warpgroups, register file re-split between them):
//   warps 0-3 / 4-7 : softmax warpgroup of slot 0 / 1.  Thread r owns query row r: it reads the
//                     score row S (fp32) from TMEM into registers and hands the S buffer back,
//                     applies scale and (partial tiles only) the mask computed from coordinates,
//                     keeps the running maximum m and sum l, writes P = 2^(S*scale*log2e - m) as
//                     bf16 into the slot's own P columns, rescales O when the maximum has grown, and
//                     at the end writes O / l and LSE.  (Algorithm 1: scale_and_mask and rowmax of
//                     the First Stage, the Second Stage, and the rescale of the Third.)
//   warp 8          : TMA producer and scheduler.  Walks the items, loads Q once per item and K_j / V_j
//                     for executed tiles only into a shared-memory ring (a tile wanted by both slots
//                     in the same step is loaded once), and publishes one command word per slot-step
//                     for the MMA issuer, with ring slots, barrier phases and release flags worked out.
//   warp 9          : MMA issuer.  Pops commands and issues S = Q K^T (both operands in shared memory)
//                     and O += P V (P from TMEM, V from shared memory) on tcgen05 with fp32
//                     accumulators in TMEM.  Its loop time is the kernel's period, so it does nothing else.
//   warps 10-11     : idle (they only keep the warpgroup complete for the register re-split).
// Tensor memory (512 columns): one S buffer that the slots use in turn (128), P of each slot
// (2 x 64), O of each slot (2 x head_dim).  S(s, t + 1) is issued before PV(s, t), so a slot's next
// scores are computed while its softmax warps still work on the current tile.  (At head_dim 64 the
// columns would allow an S buffer per slot; measured, that layout was 9 % slower.)
// Every mbarrier and queue wait is bounded; on expiry the CTA sets the status word and all roles leave.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "sm100_ptx.cuh"
#include "steel_kernel.h"
#include "steel_plan.h"

namespace steel {

constexpr int kThreads = 384;        // softmax slot 0, softmax slot 1, {producer, MMA, 2 idle warps}
// Registers per thread after the warpgroups re-split the file.  2 * 128 * kRegsSoftmax + 128 *
// kRegsOther must stay below the 65 536 registers of an SM with room to spare: setmaxnreg.inc waits,
// without any bound, until the increase can be granted.
constexpr int kRegsSoftmax = 216;
constexpr int kRegsOther = 72;
static_assert(2 * 128 * kRegsSoftmax + 128 * kRegsOther <= 65536 - 1024, "register re-split needs slack");
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr float kRescaleThreshold = 8.0f;           // lazy rescale: P stays below 2^8
constexpr int kMaxStages = 10;
constexpr int kFifoDepth = 32;
constexpr uint32_t kMaskCausal = 1u, kMaskWindow = 2u;

template <int D>
struct Cfg {
  static constexpr int kTileBytes = kTile * D * 2;  // one Q, K or V tile
  static constexpr int kBoxes = D / 64;             // 64-column (128-byte) TMA boxes per tile
  static constexpr int kBoxBytes = kTile * 128;
  static constexpr int kStages = (D == 128) ? 5 : 10;
  static constexpr int kSmemBytes = 1024 + (2 + kStages) * kTileBytes;
  // Tensor-memory columns: S (fp32, 128 columns), one buffer that the slots use in turn; P of slot s
  // (bf16 pairs, 64 columns) at kColP + 64 s; O of slot s (D columns) at kColO + D s.
  static constexpr uint32_t kColS = 0, kColP = 128, kColO = 256;
};

struct Ctrl {
  uint64_t ring_full[kMaxStages], ring_empty[kMaxStages];
  uint64_t q_full[2], q_empty[2], s_full[2], p_full[2], p_free[2], o_full[2], o_empty[2];
  uint64_t s_free;     // the softmax warps that own the S buffer's content have it in registers
  uint64_t drain;      // the MMA issuer's last commit when it leaves on an expired wait
  uint32_t fifo[kFifoDepth];  // command words from the producer to the MMA issuer (0 = empty)
  uint32_t tmem_base;
  int abort;
  long long timeout_cycles;
};

// Command word (producer -> MMA issuer): one word carries S(s, t + 1), PV(s, t) or both (the usual
// case: the first product of the next step is issued right before the second product of this one).
constexpr uint32_t kCmdValid = 1u << 0, kCmdHasPV = 1u << 1, kCmdHasS = 1u << 2, kCmdSlot1 = 1u << 3,
                   kCmdVRingShift = 4, kCmdKRingShift = 8,  // 4 bits each: ring slot of the V / K tile
                   kCmdVPhase = 1u << 12, kCmdKPhase = 1u << 13, kCmdVSkipWait = 1u << 14, kCmdKSkipWait = 1u << 15,
                   kCmdVFinal = 1u << 16, kCmdKFinal = 1u << 17,  // last user: release the ring slot
                   kCmdWaitOEmpty = 1u << 18, kCmdOEmptyPhase = 1u << 19, kCmdWaitQFull = 1u << 20,
                   kCmdQFullPhase = 1u << 21, kCmdAcc = 1u << 22, kCmdPPhase = 1u << 23, kCmdOEnd = 1u << 24,
                   kCmdQEnd = 1u << 25, kCmdWaitSFree = 1u << 26, kCmdSFreePhase = 1u << 27, kCmdExit = 1u << 31;

// Optional per-role wait accounting (compiled in with -DSTEEL_TRACE only): cycles per CTA, 32 slots.
#ifdef STEEL_TRACE
#define TRACE_T0() const long long trace_t0_ = clock64()
#define TRACE_ADD(idx) trace_acc[idx] += clock64() - trace_t0_
#define TRACE_DECL(n) long long trace_acc[n] = {}
#define TRACE_FLUSH(base, n)                                                               \
  if (p.trace)                                                                             \
    for (int i_ = 0; i_ < (n); ++i_) p.trace[size_t(blockIdx.x) * 32 + (base) + i_] = trace_acc[i_]
#else
#define TRACE_T0()
#define TRACE_ADD(idx)
#define TRACE_DECL(n)
#define TRACE_FLUSH(base, n)
#endif

__device__ __forceinline__ bool bounded_wait(uint64_t *bar, uint32_t parity, Ctrl &ctrl, int32_t *status) {
  if (mbar_test_wait(bar, parity)) return true;  // the common case: already complete, no suspension
  const long long start = clock64();
  uint32_t n = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++n & 63u) == 0) {
      if (*reinterpret_cast<volatile int *>(&ctrl.abort)) return false;
      if (clock64() - start > ctrl.timeout_cycles) {
        *reinterpret_cast<volatile int *>(&ctrl.abort) = 1;
        atomicExch(status, 5);
        return false;
      }
    }
  }
}

// One lane polls on behalf of its warp; the vote both broadcasts the outcome and orders the other
// lanes after the observation.
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, Ctrl &ctrl, int32_t *status, int lane) {
  bool ok = true;
  if (lane == 0) ok = bounded_wait(bar, parity, ctrl, status);
  return __all_sync(0xffffffffu, ok);
}

// A work item unpacked into scalars (no indexable arrays, so everything stays in registers).
struct Item {
  int batch, kv_head, head0, head1, qtile0, qtile1, lo0, lo1, hi0, hi1, n_steps, kind, j0, list_off;
  __device__ __forceinline__ int lo(int s) const { return s ? lo1 : lo0; }
  __device__ __forceinline__ int hi(int s) const { return s ? hi1 : hi0; }
  __device__ __forceinline__ int head(int s) const { return s ? head1 : head0; }
  __device__ __forceinline__ int qtile(int s) const { return s ? qtile1 : qtile0; }
  __device__ __forceinline__ bool active(int s) const { return head(s) >= 0 && hi(s) >= lo(s); }
};

__device__ __forceinline__ Item load_item(const WorkItem *items, int k) {
  const int4 *src = reinterpret_cast<const int4 *>(items + k);
  const int4 a = __ldg(src), b = __ldg(src + 1), c = __ldg(src + 2), d = __ldg(src + 3);
  Item w;
  w.batch = a.x;  w.kv_head = a.y;  w.head0 = a.z;  w.head1 = a.w;
  w.qtile0 = b.x; w.qtile1 = b.y;   w.lo0 = b.z;    w.lo1 = b.w;
  w.hi0 = c.x;    w.hi1 = c.y;      w.n_steps = c.z; w.kind = c.w;
  w.j0 = d.x;     w.list_off = d.y;
  return w;
}

// Entries {slot 0, slot 1} of step t: key-tile index plus the present bit (0 when the slot is absent).
__device__ __forceinline__ uint2 load_step(const Item &w, const StepPair *steps, int t) {
  uint2 e = make_uint2(0u, 0u);
  if (t >= w.n_steps) return e;
  if (w.kind == 0) {
    const uint32_t v = uint32_t(w.j0 + t) | kEntryPresent;
    if (w.active(0) && t >= w.lo0 && t <= w.hi0) e.x = v;
    if (w.active(1) && t >= w.lo1 && t <= w.hi1) e.y = v;
  } else {
    e = __ldg(reinterpret_cast<const uint2 *>(steps + w.list_off + t));
  }
  return e;
}

// The canonical order of an item's tensor-core operations S(s, t) = Q_s K_j^T and PV(s, t):
// O_s += P_s V_j: the order in which the producer loads tiles (at their first use) and publishes
// commands, and therefore the order in which the MMA issuer executes them.
// For each step t: first S(s, t) of slots that start at t, then for each present slot S(s, t + 1)
// followed by PV(s, t): the first product runs one step ahead of the second, so a slot's next scores
// are computed while its softmax warps still work on the current ones (they hold them in registers;
// the S buffer in TMEM is free again as soon as they are loaded).  A tile wanted by both slots in
// one step is one ring fill: slot 0 uses it first, slot 1 last (the planner guarantees lo0 <= lo1).
// `ring` counts fills.
// op(s, t, j, is_s, fill, first, last) returns false to stop.
struct RingPos {
  uint32_t slot, phase;  // next fill goes to `slot`; `phase` flips each time the ring wraps
};
struct Fill {
  uint32_t slot, phase;
};

template <int kStages, class Op>
__device__ __forceinline__ bool walk_item(const Item &w, const StepPair *steps, RingPos &ring, Op &&op) {
  Fill last_k{0, 0}, last_v{0, 0};
  auto take = [&]() {
    Fill f{ring.slot, ring.phase};
    if (++ring.slot == uint32_t(kStages)) {
      ring.slot = 0;
      ring.phase ^= 1u;
    }
    return f;
  };
  auto visit = [&](const uint2 &e, int s, int t, bool is_s) -> bool {
    const uint32_t mine = s ? e.y : e.x, other = s ? e.x : e.y;
    const bool shared = other != 0 && ((mine ^ other) & kEntryTileMask) == 0;
    Fill &last = is_s ? last_k : last_v;
    Fill f;
    bool first = true, final_use = true;
    if (s == 1 && shared) {
      f = last;
      first = false;
    } else {
      f = take();
      if (s == 0) {
        last = f;
        final_use = !shared;
      }
    }
    return op(s, t, int(mine & kEntryTileMask), is_s, f, first, final_use);
  };
  uint2 cur = load_step(w, steps, 0);
  for (int t = 0; t < w.n_steps; ++t) {
    const uint2 nxt = load_step(w, steps, t + 1);
    if (cur.x != 0 && t == w.lo0 && !visit(cur, 0, t, true)) return false;
    if (cur.y != 0 && t == w.lo1 && !visit(cur, 1, t, true)) return false;
    if (cur.x != 0) {
      if (t < w.hi0 && !visit(nxt, 0, t + 1, true)) return false;
      if (!visit(cur, 0, t, false)) return false;
    }
    if (cur.y != 0) {
      if (t < w.hi1 && !visit(nxt, 1, t + 1, true)) return false;
      if (!visit(cur, 1, t, false)) return false;
    }
    cur = nxt;
  }
  return true;
}

// ------------------------------------------------------------------------------------------------
// Bounded push into the single-producer single-consumer command queue in shared memory (the pop is
// with the MMA issuer below).
__device__ __forceinline__ bool fifo_push(Ctrl &ctrl, uint32_t &tail, uint32_t word, int32_t *status) {
  volatile uint32_t *cell = &ctrl.fifo[tail];
  if (*cell != 0) {
    const long long start = clock64();
    uint32_t n = 0;
    while (*cell != 0) {
      if ((++n & 63u) == 0) {
        if (*reinterpret_cast<volatile int *>(&ctrl.abort)) return false;
        if (clock64() - start > ctrl.timeout_cycles) {
          *reinterpret_cast<volatile int *>(&ctrl.abort) = 1;
          atomicExch(status, 5);
          return false;
        }
      }
    }
  }
  *cell = word;
  tail = (tail + 1) & (kFifoDepth - 1);
  return true;
}
// The producer is also the scheduler: it walks the items, issues the TMA loads and publishes one
// command word per slot-step (PV(s, t) fused with the S(s, t + 1) that follows it), so the MMA
// issuer's own loop stays a few instructions long.
template <int D>
__device__ void producer_role(const KernelParams &p, const CUtensorMap *map_q, const CUtensorMap *map_k,
                              const CUtensorMap *map_v, Ctrl &ctrl, uint8_t *smem_q, uint8_t *smem_ring) {
  using C = Cfg<D>;
  // measurement hook: the SM clock this CTA really ran at is cycles / nanoseconds over its run
  const bool probe = p.clock_probe != nullptr && blockIdx.x == 0;
  long long probe_c0 = 0;
  unsigned long long probe_t0 = 0;
  if (probe) {
    probe_c0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(probe_t0));
  }
  RingPos ring{0, 0};
  uint32_t n_use0 = 0, n_use1 = 0, n_sp0 = 0, n_sp1 = 0, n_s = 0, fills = 0, tail = 0, pending = 0;
  bool ok = true;
  const bool stalled = p.stall_cta == int(blockIdx.x);
  const int k_end = p.cta_begin[blockIdx.x + 1];
  for (int k = p.cta_begin[blockIdx.x]; k < k_end && ok; ++k) {
    const Item w = load_item(p.items, k);
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (!ok || !w.active(s)) continue;
      uint32_t &n_use = s ? n_use1 : n_use0;
      ok = bounded_wait(&ctrl.q_empty[s], (n_use & 1u) ^ 1u, ctrl, p.status);
      if (!ok) break;
      mbar_arrive_expect_tx(&ctrl.q_full[s], C::kTileBytes);
#pragma unroll
      for (int b = 0; b < C::kBoxes; ++b)
        tma_load_3d(smem_q + s * C::kTileBytes + b * C::kBoxBytes, map_q, &ctrl.q_full[s], b * 64,
                    w.qtile(s) * kTile, w.batch * p.heads_q + w.head(s));
      ++n_use;
    }
    if (!ok) break;
    const int z = w.batch * p.heads_kv + w.kv_head;
    ok = walk_item<C::kStages>(w, p.steps, ring, [&](int s, int t, int j, bool is_s, Fill f, bool first, bool final_use) -> bool {
      if (first) {
        if (!bounded_wait(&ctrl.ring_empty[f.slot], f.phase ^ 1u, ctrl, p.status)) return false;
        mbar_arrive_expect_tx(&ctrl.ring_full[f.slot], C::kTileBytes);
        const CUtensorMap *map = is_s ? map_k : map_v;
#pragma unroll
        for (int b = 0; b < C::kBoxes; ++b)
          tma_load_3d(smem_ring + f.slot * C::kTileBytes + b * C::kBoxBytes, map, &ctrl.ring_full[f.slot], b * 64,
                      j * kTile, z);
        ++fills;
      }
      // phase of this item's use of the slot: Q-full for S, O-empty (inverted) for PV
      const uint32_t use_phase = ((s ? n_use1 : n_use0) - 1u) & 1u;
      if (is_s) {
        // the S buffer is shared: S number n may be issued once S number n - 1 has been loaded into registers
        uint32_t part = kCmdHasS | (f.slot << kCmdKRingShift) | (f.phase ? kCmdKPhase : 0u) |
                        (first ? 0u : kCmdKSkipWait) | (final_use ? kCmdKFinal : 0u) |
                        (n_s > 0 ? kCmdWaitSFree : 0u) | (((n_s - 1u) & 1u) ? kCmdSFreePhase : 0u);
        ++n_s;
        if (t == w.lo(s)) part |= kCmdWaitQFull | (use_phase ? kCmdQFullPhase : 0u);
        if (t == w.hi(s)) part |= kCmdQEnd;
        if (t == w.lo(s)) {
          // first step of the slot: nothing of this slot to pair it with
          if (stalled) return true;  // test hook: the issuer's bounded wait for this command must expire
          return fifo_push(ctrl, tail, part | kCmdValid | (s ? kCmdSlot1 : 0u), p.status);
        }
        pending = part;  // completed by the PV(s, t - 1) that the walk visits next
        return true;
      }
      uint32_t &n_sp = s ? n_sp1 : n_sp0;
      uint32_t part = kCmdHasPV | (f.slot << kCmdVRingShift) | (f.phase ? kCmdVPhase : 0u) |
                      (first ? 0u : kCmdVSkipWait) | (final_use ? kCmdVFinal : 0u) | (t > w.lo(s) ? kCmdAcc : 0u) |
                      ((n_sp & 1u) ? kCmdPPhase : 0u);
      if (t == w.lo(s)) part |= kCmdWaitOEmpty | ((use_phase ^ 1u) ? kCmdOEmptyPhase : 0u);
      if (t == w.hi(s)) part |= kCmdOEnd;
      ++n_sp;
      const uint32_t cmd = pending | part | kCmdValid | (s ? kCmdSlot1 : 0u);
      pending = 0;
      if (stalled) return true;
      return fifo_push(ctrl, tail, cmd, p.status);
    });
  }
  if (ok) ok = fifo_push(ctrl, tail, kCmdValid | kCmdExit, p.status);
  if (probe) {
    unsigned long long t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    p.clock_probe[0] = clock64() - probe_c0;
    p.clock_probe[1] = (long long)(t1 - probe_t0);
  }
  if (!ok) {
    // leave only after the copies already issued have landed (bounded), so none writes into
    // shared memory of a later CTA: the last min(fills, stages) fills end at ring.slot - 1
    const uint32_t pending = fills < uint32_t(C::kStages) ? fills : uint32_t(C::kStages);
    uint32_t slot = ring.slot, phase = ring.phase;
    for (uint32_t e = 0; e < pending; ++e) {
      if (slot == 0) {
        slot = C::kStages;
        phase ^= 1u;
      }
      --slot;
      const long long start = clock64();
      while (!mbar_try_wait(&ctrl.ring_full[slot], phase) && clock64() - start < ctrl.timeout_cycles / 8) {
      }
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const uint32_t n_use = s ? n_use1 : n_use0;
      if (n_use) {
        const long long start = clock64();
        while (!mbar_try_wait(&ctrl.q_full[s], (n_use - 1) & 1u) && clock64() - start < ctrl.timeout_cycles / 8) {
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// tcgen05.mma, tcgen05.commit and mbarrier tests take their operands from the warp's uniform
// registers, so the issuing warp keeps everything it derives from a command word provably uniform:
// all 32 lanes run the loop and read the same queue cell, and the word is rebuilt by a warp vote
// (lane i contributes bit i).  A value loaded from shared memory by one lane is not uniform as far
// as the compiler can tell, and every operand derived from it would be copied into a uniform
// register again before each instruction that needs it.
__device__ __forceinline__ uint32_t warp_uniform(uint32_t word, int lane) {
  return __ballot_sync(0xffffffffu, (word >> lane) & 1u);
}

// Pop by the whole warp: every lane polls the same cell; the decision to leave is taken on the
// voted word, so the lanes stay together.  Lane 0 empties the cell.
__device__ __forceinline__ uint32_t fifo_pop_warp(Ctrl &ctrl, uint32_t &head, int32_t *status, int lane) {
  volatile uint32_t *cell = &ctrl.fifo[head];
  __syncwarp();
  uint32_t word = warp_uniform(*cell, lane);
  if (word == 0) {
    const long long start = clock64();
    uint32_t n = 0;
    while (true) {
      __syncwarp();
      word = warp_uniform(*cell, lane);
      if (word != 0) break;
      if ((++n & 63u) == 0) {
        const bool stop = *reinterpret_cast<volatile int *>(&ctrl.abort) != 0 || clock64() - start > ctrl.timeout_cycles;
        if (__any_sync(0xffffffffu, stop)) {
          if (lane == 0 && *reinterpret_cast<volatile int *>(&ctrl.abort) == 0) {
            *reinterpret_cast<volatile int *>(&ctrl.abort) = 1;
            atomicExch(status, 5);
          }
          return kCmdExit;
        }
      }
    }
  }
  if (lane == 0) *cell = 0;
  head = (head + 1) & (kFifoDepth - 1);
  return word;
}

template <int D>
__device__ void mma_role(const KernelParams &p, Ctrl &ctrl, uint8_t *smem_q, uint8_t *smem_ring, const int lane) {
  using C = Cfg<D>;
  const uint32_t tmem = warp_uniform(ctrl.tmem_base, lane);
  const uint32_t idesc_s = make_idesc_bf16(kTile, kTile, 0, 0);
  const uint32_t idesc_pv = make_idesc_bf16(kTile, D, 0, 1);
  const uint64_t desc_q0 = make_smem_desc(smem_u32(smem_q), 16, 1024);
  const uint64_t desc_k0 = make_smem_desc(smem_u32(smem_ring), 16, 1024);
  const uint64_t desc_v0 = make_smem_desc(smem_u32(smem_ring), C::kBoxBytes, 1024);
  uint32_t head = 0;
  bool ok = true;
  TRACE_DECL(8);
#ifdef STEEL_TRACE
  const long long role_t0 = clock64();
#endif
  uint32_t cmd = fifo_pop_warp(ctrl, head, p.status, lane);
  while (!(cmd & kCmdExit)) {
    // look at the next command now, so that its shared-memory latency hides behind this one's issue
    volatile uint32_t *next_cell = &ctrl.fifo[head];
    __syncwarp();
    const uint32_t next_raw = *next_cell;
    const uint32_t s = (cmd & kCmdSlot1) ? 1u : 0u;
    const uint32_t v_slot = (cmd >> kCmdVRingShift) & 0xFu, k_slot = (cmd >> kCmdKRingShift) & 0xFu;
    const bool has_pv = (cmd & kCmdHasPV) != 0, has_s = (cmd & kCmdHasS) != 0;
    constexpr uint32_t kRare = kCmdWaitOEmpty | kCmdWaitQFull | kCmdOEnd | kCmdQEnd;
    const uint32_t rare = cmd & kRare;
    // One elected lane does the barrier work and issues; the other lanes only keep the loop's
    // control values uniform.
    if (elect_one()) {
      TRACE_T0();
      // test the barriers the command depends on back to back, so their latencies overlap; only
      // the ones not yet complete are then waited for
      const bool need_v = has_pv && !(cmd & kCmdVSkipWait), need_k = has_s && !(cmd & kCmdKSkipWait);
      const bool need_f = has_s && (cmd & kCmdWaitSFree);
      uint64_t *s_free = &ctrl.s_free;
      bool ok_f = !need_f || mbar_test_wait(s_free, (cmd & kCmdSFreePhase) ? 1u : 0u);
      bool ok_k = !need_k || mbar_test_wait(&ctrl.ring_full[k_slot], (cmd & kCmdKPhase) ? 1u : 0u);
      bool ok_v = !need_v || mbar_test_wait(&ctrl.ring_full[v_slot], (cmd & kCmdVPhase) ? 1u : 0u);
      if (has_s) {
        // S(s, t + 1) into the shared S buffer: its previous content must be in its owners' registers
        if (rare | uint32_t(!ok_f) | uint32_t(!ok_k)) {
          if (cmd & kCmdWaitQFull)
            ok = bounded_wait(&ctrl.q_full[s], (cmd & kCmdQFullPhase) ? 1u : 0u, ctrl, p.status);
          if (ok && !ok_f) {
            TRACE_T0();
            ok = bounded_wait(s_free, (cmd & kCmdSFreePhase) ? 1u : 0u, ctrl, p.status);
            TRACE_ADD(0);
          }
          if (ok && !ok_k) {
            TRACE_T0();
            ok = bounded_wait(&ctrl.ring_full[k_slot], (cmd & kCmdKPhase) ? 1u : 0u, ctrl, p.status);
            TRACE_ADD(1);
          }
        }
        if (ok) {
          tc_fence_after();
          const uint64_t dq = desc_q0 + uint64_t((s * C::kTileBytes) >> 4);
          const uint64_t dk = desc_k0 + uint64_t((k_slot * C::kTileBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t off = uint64_t(((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            mma_ss(tmem + C::kColS, dq + off, dk + off, idesc_s, kk > 0);
          }
        }
      }
      // A commit does not return before the instructions it covers have nearly drained, so the
      // test of the next group's barrier goes between issuing this group and committing it.
      const uint32_t p_phase = (cmd & kCmdPPhase) ? 1u : 0u;
      const bool ok_p = !has_pv || mbar_test_wait(&ctrl.p_full[s], p_phase);
      if (ok && has_s) {
        tc_commit(&ctrl.s_full[s]);
        tc_commit_if(&ctrl.ring_empty[k_slot], cmd & kCmdKFinal);
        if (rare) tc_commit_if(&ctrl.q_empty[s], cmd & kCmdQEnd);
      }
      if (ok && has_pv) {
        // O_s += P_s V: P from its own TMEM columns, written by the softmax warps of slot s
        if (rare | uint32_t(!ok_p) | uint32_t(!ok_v)) {
          if (cmd & kCmdWaitOEmpty) ok = bounded_wait(&ctrl.o_empty[s], (cmd & kCmdOEmptyPhase) ? 1u : 0u, ctrl, p.status);
          if (ok && !ok_v) {
            TRACE_T0();
            ok = bounded_wait(&ctrl.ring_full[v_slot], (cmd & kCmdVPhase) ? 1u : 0u, ctrl, p.status);
            TRACE_ADD(2);
          }
          if (ok && !ok_p) {
            TRACE_T0();
            ok = bounded_wait(&ctrl.p_full[s], p_phase, ctrl, p.status);
            TRACE_ADD(3);
          }
        }
        if (ok) {
          tc_fence_after();
          const uint64_t dv = desc_v0 + uint64_t((v_slot * C::kTileBytes) >> 4);
          const uint32_t t_p = tmem + C::kColP + s * (kTile / 2);
          const uint32_t t_o = tmem + C::kColO + s * D;
          const uint32_t acc0 = (cmd & kCmdAcc) ? 1u : 0u;
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            mma_ts(t_o, t_p + kk * 8, dv + uint64_t((kk * 2048) >> 4), idesc_pv, kk > 0 ? 1u : acc0);
          tc_commit(&ctrl.p_free[s]);
          tc_commit_if(&ctrl.ring_empty[v_slot], cmd & kCmdVFinal);
          if (rare) tc_commit_if(&ctrl.o_full[s], cmd & kCmdOEnd);
        }
      }
      TRACE_ADD(5);
    }
    const uint32_t next = warp_uniform(next_raw, lane);
    if (__any_sync(0xffffffffu, !ok)) break;
    if (next != 0) {
      if (lane == 0) *next_cell = 0;
      head = (head + 1) & (kFifoDepth - 1);
      cmd = next;
    } else {
      TRACE_T0();
      cmd = fifo_pop_warp(ctrl, head, p.status, lane);
      TRACE_ADD(4);
    }
  }
#ifdef STEEL_TRACE
  trace_acc[7] = clock64() - role_t0;
  if (elect_one()) { TRACE_FLUSH(0, 8); }
#endif
  // Leaving on an expired wait: everything this warp issued must have retired before the CTA frees
  // its tensor memory, so commit to a spare barrier and wait for it (bounded).
  if (*reinterpret_cast<volatile int *>(&ctrl.abort)) {
    if (elect_one()) {
      tc_commit(&ctrl.drain);
      const long long start = clock64();
      while (!mbar_try_wait(&ctrl.drain, 0) && clock64() - start < ctrl.timeout_cycles / 8) {
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// 2^y for a pair of exponents on the FMA pipe instead of the special-function unit: y = n + f with
// n = round(y), f in [-0.5, 0.5]; 2^f by a cubic with 7.5e-5 relative error (far below bf16's
// 2^-9), scaled by adding n to the exponent field.  Inputs must be finite or -inf; they are clamped
// at -125 so the exponent field stays positive (the result is then at most 2^-125).
__device__ __forceinline__ float2 exp2_poly(float2 y) {
  const float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to the nearest integer
  y.x = fmaxf(y.x, -125.0f);
  y.y = fmaxf(y.y, -125.0f);
  const float2 t = fadd2(y, make_float2(kMagic, kMagic));
  const float2 f = fadd2(y, fadd2(make_float2(kMagic, kMagic), make_float2(-t.x, -t.y)));
  float2 q = ffma2(make_float2(5.517166907e-02f, 5.517166907e-02f), f, make_float2(2.426111222e-01f, 2.426111222e-01f));
  q = ffma2(q, f, make_float2(6.932609855e-01f, 6.932609855e-01f));
  q = ffma2(q, f, make_float2(9.999280735e-01f, 9.999280735e-01f));
  q.x = __int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23));
  q.y = __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23));
  return q;
}

// exp2 of 64 scaled scores -> 32 packed bf16x2 registers; accumulates the row sum in two lane pairs.
// With kEmu > 0, one pair in every 2^(3 - kEmu) is evaluated by exp2_poly (12.5 %, 25 %, 50 % of the
// exponentials leave the special-function unit for the FMA pipe: the counterpart of the lookup-table
// exponent the paper uses on the NPU generation that has no exponent unit).
template <int kEmu>
__device__ __forceinline__ void exp_half(const float (&x)[kTile], int base, float2 scale2, float2 neg_m2,
                                         float2 &acc_a, float2 &acc_b, uint32_t (&packed)[32]) {
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    const int e = base + 2 * i;
    float2 y0 = ffma2(make_float2(x[e], x[e + 1]), scale2, neg_m2);
    float2 y1 = ffma2(make_float2(x[e + 2], x[e + 3]), scale2, neg_m2);
    y0.x = ex2_approx(y0.x);
    y0.y = ex2_approx(y0.y);
    const bool emulate = kEmu > 0 && ((i / 2) % (1 << (3 - kEmu)) == (1 << (3 - kEmu)) - 1);
    if (emulate) {
      y1 = exp2_poly(y1);
    } else {
      y1.x = ex2_approx(y1.x);
      y1.y = ex2_approx(y1.y);
    }
    acc_a = fadd2(acc_a, y0);
    acc_b = fadd2(acc_b, y1);
    packed[i] = pack_bf16x2(y0.x, y0.y);
    packed[i + 1] = pack_bf16x2(y1.x, y1.y);
  }
}

template <int D, int kEmu>
__device__ void softmax_role(const KernelParams &p, Ctrl &ctrl, const int s, const int r) {
  using C = Cfg<D>;
  const int lane = r % 32;
  const uint32_t lane_base = uint32_t((r / 32) * 32) << 16;
  const uint32_t t_s = ctrl.tmem_base + lane_base + C::kColS;
  const uint32_t t_p = ctrl.tmem_base + lane_base + C::kColP + s * (kTile / 2);
  const uint32_t t_o = ctrl.tmem_base + lane_base + C::kColO + s * D;
  const bool causal = (p.mask_flags & kMaskCausal) != 0, windowed = (p.mask_flags & kMaskWindow) != 0;
  const int off = p.seq_kv - p.seq_q;
  const float scale_log2 = p.scale_log2;
  const float2 scale2 = make_float2(scale_log2, scale_log2);
  __nv_bfloat16 *o_base = static_cast<__nv_bfloat16 *>(p.o);
  uint32_t n_sp = 0, n_use = 0;
  TRACE_DECL(7);
#ifdef STEEL_TRACE
  const long long role_t0 = clock64();
  unsigned long long gt0;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt0));
#endif

  const int k_end = p.cta_begin[blockIdx.x + 1];
  for (int k = p.cta_begin[blockIdx.x]; k < k_end; ++k) {
    const Item w = load_item(p.items, k);
    if (w.head(s) < 0) continue;
    const int row = w.qtile(s) * kTile + r;
    const size_t out_row = (size_t(w.batch) * p.heads_q + w.head(s)) * size_t(p.seq_q) + size_t(row);
    float m_ref = -CUDART_INF_F, l = 0.0f;
    const int lo = w.lo(s), hi = w.hi(s);
    const bool active = hi >= lo;

    for (int t = lo; t <= hi; ++t) {
      // which key tile, and does it need the element-wise mask (case iii)?
      int j;
      bool partial;
      uint32_t sub = 0xF;
      if (w.kind == 0) {
        j = w.j0 + t;
        const int i0 = w.qtile(s) * kTile, i1 = min(i0 + kTile - 1, p.seq_q - 1);
        const int j0 = j * kTile, j1 = min(j0 + kTile - 1, p.seq_kv - 1);
        const bool full = (!causal || j1 <= i0 + off) && (!windowed || (i1 + off) - j0 < p.window) &&
                          (j1 - j0 + 1 == kTile);
        partial = !full;
      } else {
        const uint2 sp = __ldg(reinterpret_cast<const uint2 *>(p.steps + w.list_off + t));
        const uint32_t e = s ? sp.y : sp.x;
        j = int(e & kEntryTileMask);
        partial = (e & kEntryPartial) != 0;
        sub = (e >> kEntrySubShift) & 0xF;
      }

      bool ok;
      {
        TRACE_T0();
        ok = warp_wait(&ctrl.s_full[s], n_sp & 1u, ctrl, p.status, lane);
        TRACE_ADD(0);
      }
      if (!ok) return;
      tc_fence_after();
      TRACE_T0();

      float x[kTile];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t regs[32];
        tmem_ld32(t_s + c * 32, regs);
#pragma unroll
        for (int i = 0; i < 32; ++i) x[c * 32 + i] = __uint_as_float(regs[i]);
      }
      tc_wait_ld();
      // the scores are in registers: hand the S buffer back for the next QK^T (of either slot)
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl.s_free);
      TRACE_ADD(2);

      if (partial) {
        // visible columns of this row form one interval [c_lo, c_hi] of the tile
        const int pos = row + off, jb = j * kTile;
        int c_hi = min(kTile - 1, p.seq_kv - 1 - jb), c_lo = 0;
        if (causal) c_hi = min(c_hi, pos - jb);
        if (windowed) c_lo = max(c_lo, pos - p.window + 1 - jb);
        const uint32_t half = (sub >> (2 * (r / 64))) & 3u;  // bit 0: keys 0-63 enabled, bit 1: keys 64-127
        if (!(half & 1u)) c_lo = max(c_lo, 64);
        if (!(half & 2u)) c_hi = min(c_hi, 63);
#pragma unroll
        for (int c = 0; c < kTile; ++c) x[c] = (c >= c_lo && c <= c_hi) ? x[c] : -CUDART_INF_F;
      }

      float mx0 = fmax3(x[0], x[1], x[2]), mx1 = fmax3(x[3], x[4], x[5]);
      float mx2 = fmax3(x[6], x[7], x[8]), mx3 = fmax3(x[9], x[10], x[11]);
#pragma unroll
      for (int c = 12; c < 124; c += 8) {
        mx0 = fmax3(mx0, x[c], x[c + 1]);
        mx1 = fmax3(mx1, x[c + 2], x[c + 3]);
        mx2 = fmax3(mx2, x[c + 4], x[c + 5]);
        mx3 = fmax3(mx3, x[c + 6], x[c + 7]);
      }
      mx0 = fmax3(mx0, x[124], x[125]);
      mx1 = fmax3(mx1, x[126], x[127]);
      const float ms = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale_log2;

      if (t == lo) {
        m_ref = ms;
      } else {
        // the running maximum only has to bound the exponents: rescale O lazily
        const bool need = ms > m_ref + kRescaleThreshold;
        if (__any_sync(0xffffffffu, need)) {
          // PV(s, t - 1) accumulates into O: it must have finished
          if (!warp_wait(&ctrl.p_free[s], (n_sp - 1u) & 1u, ctrl, p.status, lane)) return;
          tc_fence_after();
          const float v = need ? ex2_approx(m_ref - ms) : 1.0f;
          l *= v;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t regs[32];
            tmem_ld32(t_o + c * 32, regs);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) regs[i] = __float_as_uint(__uint_as_float(regs[i]) * v);
            tmem_st32(t_o + c * 32, regs);
          }
          if (need) m_ref = ms;
        }
      }
      const float m_use = (m_ref == -CUDART_INF_F) ? 0.0f : m_ref;
      const float2 neg_m2 = make_float2(-m_use, -m_use);

      float2 acc_a = make_float2(0.f, 0.f), acc_b = make_float2(0.f, 0.f);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t packed[32];
        exp_half<kEmu>(x, half * 64, scale2, neg_m2, acc_a, acc_b, packed);
        if (half == 0 && t > lo) {
          // PV(s, t - 1) reads the P columns: it must have finished before they are overwritten (by
          // now it has had the whole first half of the exponentials to do so)
          if (!warp_wait(&ctrl.p_free[s], (n_sp - 1u) & 1u, ctrl, p.status, lane)) return;
          tc_fence_after();
        }
        tmem_st32(t_p + half * 32, packed);
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl.p_full[s]);
      ++n_sp;
      const float2 acc = fadd2(acc_a, acc_b);
      // The polynomial path returns 2^-125 rather than 0 for a masked (-inf) score: a row that has
      // not seen a visible key yet (m = -inf) must keep l = 0 exactly, so that it ends as O = 0.
      if (kEmu == 0 || m_ref != -CUDART_INF_F) l += acc.x + acc.y;
      TRACE_ADD(3);
    }

    // epilogue: O / l and LSE = ln2 * (m + log2 l)
    if (active) {
      bool ok;
      {
        TRACE_T0();
        ok = warp_wait(&ctrl.o_full[s], n_use & 1u, ctrl, p.status, lane);
        TRACE_ADD(1);
      }
      if (!ok) return;
      ++n_use;
      tc_fence_after();
      TRACE_T0();
      const float inv = l > 0.0f ? 1.0f / l : 0.0f;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t regs[32];
        tmem_ld32(t_o + c * 32, regs);
        tc_wait_ld();
        if (row < p.seq_q) {
          uint4 *dst = reinterpret_cast<uint4 *>(o_base + out_row * D + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16x2(__uint_as_float(regs[8 * i + 0]) * inv, __uint_as_float(regs[8 * i + 1]) * inv);
            v.y = pack_bf16x2(__uint_as_float(regs[8 * i + 2]) * inv, __uint_as_float(regs[8 * i + 3]) * inv);
            v.z = pack_bf16x2(__uint_as_float(regs[8 * i + 4]) * inv, __uint_as_float(regs[8 * i + 5]) * inv);
            v.w = pack_bf16x2(__uint_as_float(regs[8 * i + 6]) * inv, __uint_as_float(regs[8 * i + 7]) * inv);
            dst[i] = v;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl.o_empty[s]);
      if (p.lse != nullptr && row < p.seq_q)
        p.lse[out_row] = l > 0.0f ? 0.6931471805599453f * (m_ref + log2f(l)) : -CUDART_INF_F;
      TRACE_ADD(4);
    } else if (row < p.seq_q) {
      // no key tile is visible to this query tile
      uint4 *dst = reinterpret_cast<uint4 *>(o_base + out_row * D);
#pragma unroll
      for (int i = 0; i < D / 8; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
      if (p.lse != nullptr) p.lse[out_row] = -CUDART_INF_F;
    }
  }
#ifdef STEEL_TRACE
  trace_acc[6] = clock64() - role_t0;
  if (r == 0) {
    unsigned long long gt1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt1));
    if (p.trace && s == 0) p.trace[size_t(blockIdx.x) * 32 + 15] = (long long)(gt1 - gt0);
    TRACE_FLUSH(16 + 8 * s, 7);
  }
#endif
}

// ------------------------------------------------------------------------------------------------
template <int D, int kEmu>
__global__ void __launch_bounds__(kThreads, 1)
steel_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const __grid_constant__ KernelParams p) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Ctrl ctrl;
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_q = smem;
  uint8_t *smem_ring = smem + 2 * C::kTileBytes;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::kStages; ++i) {
      mbar_init(&ctrl.ring_full[i], 1);
      mbar_init(&ctrl.ring_empty[i], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&ctrl.q_full[s], 1);
      mbar_init(&ctrl.q_empty[s], 1);
      mbar_init(&ctrl.s_full[s], 1);
      mbar_init(&ctrl.p_full[s], 4);  // one arrival per softmax warp
      mbar_init(&ctrl.p_free[s], 1);
      mbar_init(&ctrl.o_full[s], 1);
      mbar_init(&ctrl.o_empty[s], 4);
    }
    mbar_init(&ctrl.s_free, 4);
    mbar_init(&ctrl.drain, 1);
    for (int i = 0; i < kFifoDepth; ++i) ctrl.fifo[i] = 0;
    ctrl.abort = 0;
    ctrl.timeout_cycles = p.timeout_cycles;
    fence_barrier_init();
  }
  if (warp == kProducerWarp && lane == 0) {
    prefetch_tensormap(&map_q);
    prefetch_tensormap(&map_k);
    prefetch_tensormap(&map_v);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&ctrl.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (warp < 8) {
    setmaxnreg_inc<kRegsSoftmax>();
    softmax_role<D, kEmu>(p, ctrl, warp / 4, threadIdx.x % kTile);
  } else {
    setmaxnreg_dec<kRegsOther>();
    if (warp == kProducerWarp) {
      if (lane == 0) producer_role<D>(p, &map_q, &map_k, &map_v, ctrl, smem_q, smem_ring);
    } else if (warp == kMmaWarp) {
      mma_role<D>(p, ctrl, smem_q, smem_ring, lane);
    }
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(ctrl.tmem_base, 512);
}

namespace {

template <int D, int kEmu>
cudaError_t configure_one() {
  return cudaFuncSetAttribute(steel_attn_kernel<D, kEmu>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<D>::kSmemBytes);
}

template <int D, int kEmu>
void launch_one(const CUtensorMap &map_q, const CUtensorMap &map_k, const CUtensorMap &map_v,
                const KernelParams &params, int grid, cudaStream_t stream) {
  steel_attn_kernel<D, kEmu><<<grid, kThreads, Cfg<D>::kSmemBytes, stream>>>(map_q, map_k, map_v, params);
}

template <int D>
void launch_dim(int exp_emulation, const CUtensorMap &map_q, const CUtensorMap &map_k, const CUtensorMap &map_v,
                const KernelParams &params, int grid, cudaStream_t stream) {
  switch (exp_emulation) {
    case 1: launch_one<D, 1>(map_q, map_k, map_v, params, grid, stream); break;
    case 2: launch_one<D, 2>(map_q, map_k, map_v, params, grid, stream); break;
    case 3: launch_one<D, 3>(map_q, map_k, map_v, params, grid, stream); break;
    default: launch_one<D, 0>(map_q, map_k, map_v, params, grid, stream); break;
  }
}

}  // namespace

cudaError_t configure_kernels() {
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = configure_one<128, 0>();
  if (e == cudaSuccess) e = configure_one<128, 1>();
  if (e == cudaSuccess) e = configure_one<128, 2>();
  if (e == cudaSuccess) e = configure_one<128, 3>();
  if (e == cudaSuccess) e = configure_one<64, 0>();
  if (e == cudaSuccess) e = configure_one<64, 1>();
  if (e == cudaSuccess) e = configure_one<64, 2>();
  if (e == cudaSuccess) e = configure_one<64, 3>();
  return e;
}

cudaError_t launch_attention(int head_dim, int exp_emulation, const CUtensorMap &map_q, const CUtensorMap &map_k,
                             const CUtensorMap &map_v, const KernelParams &params, int grid, cudaStream_t stream) {
  if (head_dim == 128)
    launch_dim<128>(exp_emulation, map_q, map_k, map_v, params, grid, stream);
  else
    launch_dim<64>(exp_emulation, map_q, map_k, map_v, params, grid, stream);
  return cudaGetLastError();
}

}  // namespace steel
