// Fused block-sparse attention kernel for sm_100a (paper Algorithm 1 on one persistent CTA per SM).
//
// A CTA processes work items; an item is one or two query tiles (128 rows each, "slots") that walk
// the same sequence of key-tile steps.  Roles:
//   warps 0-3 / 4-7 : softmax warpgroup of slot 0 / 1.  Thread r owns query row r: it reads the
//                     score row S (fp32) from TMEM, applies scale and (partial tiles only) the mask
//                     computed from coordinates, keeps the running maximum m and sum l, writes
//                     P = 2^(S*scale*log2e - m) as bf16 back into TMEM over S, rescales O when the
//                     maximum has grown, and at the end writes O / l and LSE.  (Algorithm 1, First
//                     Stage's scale_and_mask and rowmax, Second Stage, and the rescale of the Third.)
//   warp 8          : TMA producer.  Loads Q once per item and K_j / V_j for executed tiles only into
//                     a shared-memory ring; a tile wanted by both slots in the same step is loaded once.
//   warp 9          : MMA issuer.  S = Q K^T (both operands in shared memory) and O += P V (P from
//                     TMEM, V from shared memory) on tcgen05 with fp32 accumulators in TMEM.
// All three walk an item's steps with the same generator (walk_item), so ring positions agree
// without communication.  Every mbarrier wait is bounded; on expiry the CTA sets the status word
// and all roles leave.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "sm100_ptx.cuh"
#include "steel_kernel.h"
#include "steel_plan.h"

namespace steel {

constexpr int kThreads = 320;
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr long long kTimeoutCycles = 4000000000ll;  // about two seconds
constexpr float kRescaleThreshold = 8.0f;           // lazy rescale: P stays below 2^8
constexpr int kMaxStages = 10;
constexpr uint32_t kMaskCausal = 1u, kMaskWindow = 2u;

template <int D>
struct Cfg {
  static constexpr int kTileBytes = kTile * D * 2;  // one Q, K or V tile
  static constexpr int kBoxes = D / 64;             // 64-column (128-byte) TMA boxes per tile
  static constexpr int kBoxBytes = kTile * 128;
  static constexpr int kStages = (D == 128) ? 5 : 10;
  static constexpr int kSmemBytes = 1024 + (2 + kStages) * kTileBytes;
  static constexpr uint32_t kColS = 0;    // S of slot s at columns kColS + 128 s (P aliases its first 64)
  static constexpr uint32_t kColO = 256;  // O of slot s at columns kColO + D s
};

struct Ctrl {
  uint64_t ring_full[kMaxStages], ring_empty[kMaxStages];
  uint64_t q_full[2], q_empty[2], s_full[2], p_full[2], o_full[2], o_empty[2];
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ bool bounded_wait(uint64_t *bar, uint32_t parity, Ctrl &ctrl, int32_t *status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  uint32_t n = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++n & 63u) == 0) {
      if (*reinterpret_cast<volatile int *>(&ctrl.abort)) return false;
      if (clock64() - start > kTimeoutCycles) {
        *reinterpret_cast<volatile int *>(&ctrl.abort) = 1;
        atomicExch(status, 5);
        return false;
      }
    }
  }
}

__device__ __forceinline__ WorkItem load_item(const WorkItem *items, int k) {
  WorkItem w;
  const int4 *src = reinterpret_cast<const int4 *>(items + k);
  int4 *dst = reinterpret_cast<int4 *>(&w);
#pragma unroll
  for (int i = 0; i < 4; ++i) dst[i] = __ldg(src + i);
  return w;
}

__device__ __forceinline__ bool slot_active(const WorkItem &w, int s) { return w.head[s] >= 0 && w.hi[s] >= w.lo[s]; }

// Entries {slot 0, slot 1} of step t: key-tile index plus the present bit (0 when the slot is absent).
__device__ __forceinline__ uint2 load_step(const WorkItem &w, const StepPair *steps, int t) {
  uint2 e = make_uint2(0u, 0u);
  if (t >= w.n_steps) return e;
  if (w.kind == 0) {
    uint32_t v = uint32_t(w.j0 + t) | kEntryPresent;
    if (slot_active(w, 0) && t >= w.lo[0] && t <= w.hi[0]) e.x = v;
    if (slot_active(w, 1) && t >= w.lo[1] && t <= w.hi[1]) e.y = v;
  } else {
    e = __ldg(reinterpret_cast<const uint2 *>(steps + w.list_off + t));
  }
  return e;
}

// The canonical order of an item's tensor-core operations, shared by the producer (which loads a
// tile at its first use) and the MMA issuer.  For each step t: first S(s, t) of slots that start
// at t, then for each present slot PV(s, t) followed by S(s, t + 1).  `entry` numbers ring fills;
// a tile wanted by both slots in one step is filled once (slot 0 first, slot 1 last).
template <class OpS, class OpPV>
__device__ __forceinline__ void walk_item(const WorkItem &w, const StepPair *steps, uint32_t &ring_pos, OpS &&op_s,
                                          OpPV &&op_pv, bool &ok) {
  uint32_t last_k = 0, last_v = 0;
  uint2 cur = load_step(w, steps, 0), nxt;
  auto ent = [](const uint2 &e, int s) { return s == 0 ? e.x : e.y; };
  auto visit = [&](const uint2 &e, int s, int t, bool is_s) {
    const uint32_t mine = ent(e, s), other = ent(e, 1 - s);
    const bool shared = other != 0 && ((mine ^ other) & kEntryTileMask) == 0;
    uint32_t &last = is_s ? last_k : last_v;
    uint32_t entry;
    bool first, final_use;
    if (s == 0) {
      entry = ring_pos++;
      last = entry;
      first = true;
      final_use = !shared;
    } else if (shared) {
      entry = last;
      first = false;
      final_use = true;
    } else {
      entry = ring_pos++;
      first = true;
      final_use = true;
    }
    const int j = int(mine & kEntryTileMask);
    if (is_s) ok = op_s(s, t, j, entry, first, final_use);
    else ok = op_pv(s, t, j, entry, first, final_use);
  };
  for (int t = 0; t < w.n_steps && ok; ++t) {
    nxt = load_step(w, steps, t + 1);
#pragma unroll
    for (int s = 0; s < 2; ++s)
      if (ok && ent(cur, s) != 0 && t == w.lo[s]) visit(cur, s, t, true);
#pragma unroll
    for (int s = 0; s < 2; ++s)
      if (ok && ent(cur, s) != 0) {
        visit(cur, s, t, false);
        if (ok && t < w.hi[s]) visit(nxt, s, t + 1, true);
      }
    cur = nxt;
  }
}

// ------------------------------------------------------------------------------------------------
template <int D>
__device__ void producer_role(const KernelParams &p, const CUtensorMap *map_q, const CUtensorMap *map_k,
                              const CUtensorMap *map_v, Ctrl &ctrl, uint8_t *smem_q, uint8_t *smem_ring) {
  using C = Cfg<D>;
  uint32_t ring_pos = 0, n_use[2] = {0, 0}, q_issued[2] = {0, 0};
  bool ok = true;
  auto load_tile = [&](const CUtensorMap *map, int j, int z, uint32_t entry) -> bool {
    const uint32_t slot = entry % C::kStages, fill = entry / C::kStages;
    if (!bounded_wait(&ctrl.ring_empty[slot], (fill & 1u) ^ 1u, ctrl, p.status)) return false;
    mbar_arrive_expect_tx(&ctrl.ring_full[slot], C::kTileBytes);
#pragma unroll
    for (int b = 0; b < C::kBoxes; ++b)
      tma_load_3d(smem_ring + slot * C::kTileBytes + b * C::kBoxBytes, map, &ctrl.ring_full[slot], b * 64, j * kTile, z);
    return true;
  };
  const int k_end = p.cta_begin[blockIdx.x + 1];
  for (int k = p.cta_begin[blockIdx.x]; k < k_end && ok; ++k) {
    const WorkItem w = load_item(p.items, k);
    for (int s = 0; s < 2 && ok; ++s) {
      if (!slot_active(w, s)) continue;
      ok = bounded_wait(&ctrl.q_empty[s], (n_use[s] & 1u) ^ 1u, ctrl, p.status);
      if (!ok) break;
      mbar_arrive_expect_tx(&ctrl.q_full[s], C::kTileBytes);
#pragma unroll
      for (int b = 0; b < C::kBoxes; ++b)
        tma_load_3d(smem_q + s * C::kTileBytes + b * C::kBoxBytes, map_q, &ctrl.q_full[s], b * 64,
                    w.qtile[s] * kTile, w.batch * p.heads_q + w.head[s]);
      ++n_use[s];
      q_issued[s] = n_use[s];
    }
    const int z = w.batch * p.heads_kv + w.kv_head;
    walk_item(
        w, p.steps, ring_pos,
        [&](int, int, int j, uint32_t entry, bool first, bool) { return first ? load_tile(map_k, j, z, entry) : true; },
        [&](int, int, int j, uint32_t entry, bool first, bool) { return first ? load_tile(map_v, j, z, entry) : true; },
        ok);
  }
  if (!ok) {
    // leave only after the copies already issued have landed (bounded), so none writes into
    // shared memory of a later CTA
    const uint32_t first = ring_pos > uint32_t(C::kStages) ? ring_pos - C::kStages : 0;
    for (uint32_t e = first; e < ring_pos; ++e) {
      const long long start = clock64();
      while (!mbar_try_wait(&ctrl.ring_full[e % C::kStages], (e / C::kStages) & 1u) && clock64() - start < kTimeoutCycles / 8) {
      }
    }
    for (int s = 0; s < 2; ++s)
      if (q_issued[s]) {
        const long long start = clock64();
        while (!mbar_try_wait(&ctrl.q_full[s], (q_issued[s] - 1) & 1u) && clock64() - start < kTimeoutCycles / 8) {
        }
      }
  }
}

// ------------------------------------------------------------------------------------------------
template <int D>
__device__ void mma_role(const KernelParams &p, Ctrl &ctrl, uint8_t *smem_q, uint8_t *smem_ring) {
  using C = Cfg<D>;
  const uint32_t tmem = ctrl.tmem_base;
  const uint32_t idesc_s = make_idesc_bf16(kTile, kTile, 0, 0);
  const uint32_t idesc_pv = make_idesc_bf16(kTile, D, 0, 1);
  // K-major operands (Q, K): 8-row groups 1024 bytes apart.  V is MN-major: 8-key groups 1024
  // bytes apart, the next 64 columns of head_dim one box further.
  const uint64_t desc_q0 = make_smem_desc(smem_u32(smem_q), 16, 1024);
  const uint64_t desc_k0 = make_smem_desc(smem_u32(smem_ring), 16, 1024);
  const uint64_t desc_v0 = make_smem_desc(smem_u32(smem_ring), C::kBoxBytes, 1024);
  uint32_t ring_pos = 0, n_sp[2] = {0, 0}, n_use[2] = {0, 0};
  bool ok = true;
  const int k_end = p.cta_begin[blockIdx.x + 1];
  for (int k = p.cta_begin[blockIdx.x]; k < k_end && ok; ++k) {
    const WorkItem w = load_item(p.items, k);
    walk_item(
        w, p.steps, ring_pos,
        [&](int s, int t, int, uint32_t entry, bool, bool final_use) -> bool {
          const uint32_t slot = entry % C::kStages, fill = entry / C::kStages;
          if (t == w.lo[s] && !bounded_wait(&ctrl.q_full[s], n_use[s] & 1u, ctrl, p.status)) return false;
          if (!bounded_wait(&ctrl.ring_full[slot], fill & 1u, ctrl, p.status)) return false;
          tc_fence_after();
          const uint64_t dq = desc_q0 + uint64_t((s * C::kTileBytes) >> 4);
          const uint64_t dk = desc_k0 + uint64_t((slot * C::kTileBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t off = uint64_t(((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            mma_ss(tmem + C::kColS + s * kTile, dq + off, dk + off, idesc_s, kk > 0);
          }
          tc_commit(&ctrl.s_full[s]);
          if (final_use) tc_commit(&ctrl.ring_empty[slot]);
          if (t == w.hi[s]) tc_commit(&ctrl.q_empty[s]);
          return true;
        },
        [&](int s, int t, int, uint32_t entry, bool, bool final_use) -> bool {
          const uint32_t slot = entry % C::kStages, fill = entry / C::kStages;
          if (!bounded_wait(&ctrl.p_full[s], n_sp[s] & 1u, ctrl, p.status)) return false;
          ++n_sp[s];
          if (t == w.lo[s] && !bounded_wait(&ctrl.o_empty[s], (n_use[s] & 1u) ^ 1u, ctrl, p.status)) return false;
          if (!bounded_wait(&ctrl.ring_full[slot], fill & 1u, ctrl, p.status)) return false;
          tc_fence_after();
          const uint64_t dv = desc_v0 + uint64_t((slot * C::kTileBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            mma_ts(tmem + C::kColO + s * D, tmem + C::kColS + s * kTile + kk * 8, dv + uint64_t((kk * 2048) >> 4),
                   idesc_pv, (t > w.lo[s] || kk > 0) ? 1u : 0u);
          if (final_use) tc_commit(&ctrl.ring_empty[slot]);
          if (t == w.hi[s]) {
            tc_commit(&ctrl.o_full[s]);
            ++n_use[s];
          }
          return true;
        },
        ok);
  }
}

// ------------------------------------------------------------------------------------------------
template <int D>
__device__ void softmax_role(const KernelParams &p, Ctrl &ctrl, const int s, const int r) {
  using C = Cfg<D>;
  const uint32_t lane_base = uint32_t((r / 32) * 32) << 16;
  const uint32_t t_s = ctrl.tmem_base + lane_base + C::kColS + s * kTile;
  const uint32_t t_o = ctrl.tmem_base + lane_base + C::kColO + s * D;
  const bool causal = (p.mask_flags & kMaskCausal) != 0, windowed = (p.mask_flags & kMaskWindow) != 0;
  const int off = p.seq_kv - p.seq_q;
  const float scale_log2 = p.scale_log2;
  __nv_bfloat16 *o_base = static_cast<__nv_bfloat16 *>(p.o);
  uint32_t n_sp = 0, n_use = 0;

  const int k_end = p.cta_begin[blockIdx.x + 1];
  for (int k = p.cta_begin[blockIdx.x]; k < k_end; ++k) {
    const WorkItem w = load_item(p.items, k);
    if (w.head[s] < 0) continue;
    const int row = w.qtile[s] * kTile + r;
    const size_t out_row = (size_t(w.batch) * p.heads_q + w.head[s]) * size_t(p.seq_q) + size_t(row);
    float m_ref = -CUDART_INF_F, l = 0.0f;
    const bool active = w.hi[s] >= w.lo[s];

    for (int t = w.lo[s]; t <= w.hi[s]; ++t) {
      // which key tile, and does it need the element-wise mask (case iii)?
      int j;
      bool partial;
      uint32_t sub = 0xF;
      if (w.kind == 0) {
        j = w.j0 + t;
        const int i0 = w.qtile[s] * kTile, i1 = min(i0 + kTile - 1, p.seq_q - 1);
        const int j0 = j * kTile, j1 = min(j0 + kTile - 1, p.seq_kv - 1);
        const bool full = (!causal || j1 <= i0 + off) && (!windowed || (i1 + off) - j0 < p.window) &&
                          (j1 - j0 + 1 == kTile);
        partial = !full;
      } else {
        const StepPair sp = p.steps[w.list_off + t];
        const uint32_t e = sp.e[s];
        j = int(e & kEntryTileMask);
        partial = (e & kEntryPartial) != 0;
        sub = (e >> kEntrySubShift) & 0xF;
      }

      bool ok = bounded_wait(&ctrl.s_full[s], n_sp & 1u, ctrl, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++n_sp;
      tc_fence_after();

      float x[kTile];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t regs[32];
        tmem_ld32(t_s + c * 32, regs);
#pragma unroll
        for (int i = 0; i < 32; ++i) x[c * 32 + i] = __uint_as_float(regs[i]);
      }
      tc_wait_ld();

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

      float mx0 = x[0], mx1 = x[1], mx2 = x[2], mx3 = x[3];
#pragma unroll
      for (int c = 4; c < kTile; c += 4) {
        mx0 = fmaxf(mx0, x[c]);
        mx1 = fmaxf(mx1, x[c + 1]);
        mx2 = fmaxf(mx2, x[c + 2]);
        mx3 = fmaxf(mx3, x[c + 3]);
      }
      const float ms = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale_log2;

      if (t == w.lo[s]) {
        m_ref = ms;
      } else {
        // the running maximum only has to bound the exponents: rescale O lazily
        const bool need = ms > m_ref + kRescaleThreshold;
        if (__any_sync(0xffffffffu, need)) {
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

      float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t packed[32];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const int e = c * 64 + 2 * i;
          const float p0 = ex2_approx(fmaf(x[e], scale_log2, -m_use));
          const float p1 = ex2_approx(fmaf(x[e + 1], scale_log2, -m_use));
          const float p2 = ex2_approx(fmaf(x[e + 2], scale_log2, -m_use));
          const float p3 = ex2_approx(fmaf(x[e + 3], scale_log2, -m_use));
          l0 += p0;
          l1 += p1;
          l2 += p2;
          l3 += p3;
          packed[i] = pack_bf16x2(p0, p1);
          packed[i + 1] = pack_bf16x2(p2, p3);
        }
        tmem_st32(t_s + c * 32, packed);
      }
      l += (l0 + l1) + (l2 + l3);
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(&ctrl.p_full[s]);
    }

    // epilogue: O / l and LSE = ln2 * (m + log2 l)
    if (active) {
      bool ok = bounded_wait(&ctrl.o_full[s], n_use & 1u, ctrl, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++n_use;
      tc_fence_after();
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
      mbar_arrive(&ctrl.o_empty[s]);
      if (p.lse != nullptr && row < p.seq_q)
        p.lse[out_row] = l > 0.0f ? 0.6931471805599453f * (m_ref + log2f(l)) : -CUDART_INF_F;
    } else if (row < p.seq_q) {
      // no key tile is visible to this query tile
      uint4 *dst = reinterpret_cast<uint4 *>(o_base + out_row * D);
#pragma unroll
      for (int i = 0; i < D / 8; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
      if (p.lse != nullptr) p.lse[out_row] = -CUDART_INF_F;
    }
  }
}

// ------------------------------------------------------------------------------------------------
template <int D>
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
      mbar_init(&ctrl.p_full[s], kTile);
      mbar_init(&ctrl.o_full[s], 1);
      mbar_init(&ctrl.o_empty[s], kTile);
    }
    ctrl.abort = 0;
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
    softmax_role<D>(p, ctrl, warp / 4, threadIdx.x % kTile);
  } else if (warp == kProducerWarp) {
    if (lane == 0) producer_role<D>(p, &map_q, &map_k, &map_v, ctrl, smem_q, smem_ring);
  } else {
    if (lane == 0) mma_role<D>(p, ctrl, smem_q, smem_ring);
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(ctrl.tmem_base, 512);
}

cudaError_t configure_kernels() {
  cudaError_t e = cudaFuncSetAttribute(steel_attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Cfg<128>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(steel_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<64>::kSmemBytes);
}

cudaError_t launch_attention(int head_dim, const CUtensorMap &map_q, const CUtensorMap &map_k,
                             const CUtensorMap &map_v, const KernelParams &params, int grid, cudaStream_t stream) {
  if (head_dim == 128)
    steel_attn_kernel<128><<<grid, kThreads, Cfg<128>::kSmemBytes, stream>>>(map_q, map_k, map_v, params);
  else
    steel_attn_kernel<64><<<grid, kThreads, Cfg<64>::kSmemBytes, stream>>>(map_q, map_k, map_v, params);
  return cudaGetLastError();
}

}  // namespace steel
