// Compression policies in which rows are owned per UNIT (sm_100a): a unit is one
// KV head (TOVA-head, H2O head-wise) or the whole layer (H2O layer-wise).
//
//   TOVA-head (Section 4; appendix ablation): every head scores the rows by its own
//       attention weights and drops its own lowest one, so heads come to hold
//       different tokens.
//   H2O (Section 4.1): the `recent` most recent tokens always stay; among the older
//       rows the one whose weight, summed over all the steps it has been in the
//       state, is lowest goes.  Layer-wise the weights are averaged over all query
//       heads first, head-wise every head keeps its own sums and its own rows.
//
// Under grouped-query attention the unit that owns rows is the KV head; its score
// for a row is the mean weight of the query heads that read it.
//
// The streaming kernels are the ones of the layer policy (logits to the fp32
// scratch, per-chunk or per-head soft-max statistics); only the stage that picks
// the victim differs: one thread block per (unit, sequence) rebuilds the global
// (max, sum) of the unit's heads, scores every candidate in a fixed order,
// updates the accumulated scores (H2O), takes the arg-min - lowest slot on ties,
// the new token counting as slot `capacity` - and puts the new token's key, value,
// position and first score into the freed slot of the unit's KV heads.  Where the
// (unit, sequence) pairs are too few to fill the GPU (H2O layer-wise: one unit),
// the candidates of a pair are cut into slices, one thread block each; the block
// that finishes last (a ticket counter) merges the slices' minima in slice order
// and does the insert, so no block ever waits for another.
#pragma once

#include "tova_kernels.cuh"

namespace tova {

constexpr int POLICY_TOVA_HEAD = 2, POLICY_H2O_LAYER = 3, POLICY_H2O_HEAD = 4;
constexpr int UNIT_THREADS = 512;
constexpr int UNIT_MAX_SLICES = 8;

struct UnitPartial {   // a slice's arg-min: value, slot, position held there; the new token's weight (its slice only)
  float val;
  int32_t idx, pos;
  float wnew;
};

struct UnitParams {
  int32_t* table;     // [B,U,cap] position held by every slot of every unit
  float* acc;         // [B,U,cap] accumulated scores (H2O)
  int32_t units;      // U: 1 (layer) or Hkv (one unit per KV head)
  int32_t recent;     // H2O: candidates fewer than `recent` positions behind the new token are never dropped
  int32_t h2o;        // scores accumulate over the steps
  UnitPartial* part;  // [B,U,UNIT_MAX_SLICES] slice minima (used when gridDim.z > 1)
  int32_t* ticket;    // [B,U] blocks of the pair that have finished this step; zero between steps
};

// grid = (U, B, slices), block = UNIT_THREADS.  Dynamic shared memory: one float per head of the unit.
template <typename T, int D>
__global__ void __launch_bounds__(UNIT_THREADS) tova_unit_policy_kernel(const StepParams p, const UnitParams up) {
  extern __shared__ __align__(16) float usm[];
  const int u = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NW = UNIT_THREADS / 32;
  const int nh = (up.units == 1) ? p.H : p.G;           // query heads whose weights this unit averages
  const int h0 = (up.units == 1) ? 0 : u * p.G;
  const int kv0 = (up.units == 1) ? 0 : u, kv_n = (up.units == 1) ? p.Hkv : 1;
  float* hc = usm;                                       // [nh] -max2 - log2(sum * nh)
  __shared__ float red_v[NW];
  __shared__ int red_i[NW];
  __shared__ int red_p[NW];
  __shared__ float s_wnew;
  __shared__ int s_victim;
  __shared__ int s_last;
  const int nz = gridDim.z, z = blockIdx.z;
  const int slice = (p.n + 1 + nz - 1) / nz;             // candidates 0..n (n = the new token) in nz slices
  const int j_lo = z * slice, j_hi = min(p.n + 1, j_lo + slice);
  const bool owns_new = (p.n >= j_lo && p.n < j_hi);     // exactly one slice holds the new token

  const int pos_t = *p.cur_pos;
  int32_t* table = up.table + ((size_t)b * up.units + u) * p.cap;
  float* acc = up.acc + ((size_t)b * up.units + u) * p.cap;

  // ---- global (max, sum) of every head of the unit --------------------------------
  if (p.fuse_out) {
    for (int h = tid; h < nh; h += UNIT_THREADS) {
      const float2 e = p.head_ml[(size_t)b * p.H + h0 + h];
      hc[h] = -e.x - __log2f(e.y * (float)nh);
    }
  } else {
    const int np = p.n_chunks + 1;                       // the chunks, then the new token
    for (int h = warp; h < nh; h += NW) {
      const float2* ml = p.part_ml + ((size_t)b * p.H + h0 + h) * p.pc;
      float M = -INFINITY;
      for (int i = lane; i < np; i += 32) M = fmaxf(M, ml[i].x);
      M = warp_max(M);
      float L = 0.f;
      for (int i = lane; i < np; i += 32) L = fmaf(ml[i].y, exp2_diff(ml[i].x, M), L);
      L = warp_sum(L);
      if (lane == 0) hc[h] = -M - __log2f(L * (float)nh);
    }
  }
  __syncthreads();

  // ---- score of every candidate: mean over the unit's heads of the soft-max weight --
  const float* lg = p.logits + ((size_t)b * p.H + h0) * p.ld;
  float val = INFINITY;
  int idx = 0x7fffffff, cpos = pos_t;
  for (int j = j_lo + tid; j < j_hi; j += UNIT_THREADS) {
    float w = 0.f;
    {
      int h = 0;
      for (; h + 7 < nh; h += 8) {          // eight heads' logits requested before the first is used
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = lg[(size_t)(h + e) * p.ld + j] + hc[h + e];
#pragma unroll
        for (int e = 0; e < 8; ++e) w += exp2f(x[e]);
      }
      for (; h < nh; ++h) w += exp2f(lg[(size_t)h * p.ld + j] + hc[h]);
    }
    float key = w;
    const int pj = (j < p.n) ? table[j] : pos_t;
    if (up.h2o && j < p.n) {             // the row's weight at this step joins its sum before the choice
      key = acc[j] + w;
      acc[j] = key;
    }
    if (j == p.n) s_wnew = w;            // the new token's score so far: its weight at this step
    if (up.h2o && pos_t - pj < up.recent) key = INFINITY;   // inside the recent window
    if (key < val) { val = key; idx = j; cpos = pj; }       // j ascends: strict < keeps the lowest slot
  }

  if (!p.do_evict) {                     // g(t) = min(t, k) not reached: the new token takes the next free row
    if (!owns_new) return;               // (the other slices only had scores to add)
    __syncthreads();
    for (int i = tid; i < kv_n * (D * (int)sizeof(T) / 16); i += UNIT_THREADS) {
      constexpr int RB16 = D * (int)sizeof(T) / 16;
      const int kv = kv0 + i / RB16;
      const size_t dst = (((size_t)b * p.Hkv + kv) * p.cap + p.n) * RB16 + i % RB16;
      const size_t src = ((size_t)b * p.Hkv + kv) * RB16 + i % RB16;
      static_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[src];
      static_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[src];
    }
    if (tid == 0) {
      table[p.n] = pos_t;
      if (up.h2o) acc[p.n] = s_wnew;
      if (u == 0) p.len[b] = p.n + 1;
      if (p.evicted) p.evicted[(size_t)b * up.units + u] = -1;
    }
    return;
  }

  // ---- arg-min of the block: lowest (value, slot) ------------------------------------
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    const int op = __shfl_xor_sync(0xffffffffu, cpos, o);
    if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; cpos = op; }
  }
  if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; red_p[warp] = cpos; }
  __syncthreads();                       // also: every accumulated score is stored before one is replaced
  if (tid == 0) {
    for (int w = 1; w < NW; ++w)
      if (red_v[w] < val || (red_v[w] == val && red_i[w] < idx)) { val = red_v[w]; idx = red_i[w]; cpos = red_p[w]; }
    s_last = 1;
    if (nz > 1) {
      // This slice's minimum goes to global memory; the block that draws the last ticket merges them all.
      UnitPartial* part = up.part + ((size_t)b * up.units + u) * UNIT_MAX_SLICES;
      int32_t* ticket = up.ticket + (size_t)b * up.units + u;
      UnitPartial mine;
      mine.val = val; mine.idx = idx; mine.pos = cpos; mine.wnew = owns_new ? s_wnew : 0.f;
      part[z] = mine;
      __threadfence();                   // the partial and (through the barrier above) the block's scores, before the ticket
      s_last = (atomicAdd(ticket, 1) == nz - 1);
      if (s_last) {
        __threadfence();
        val = INFINITY; idx = 0x7fffffff; cpos = pos_t;
        for (int q = 0; q < nz; ++q) {   // slice order = slot order: strict < keeps the lowest slot
          const volatile UnitPartial* o = part + q;
          const float ov = o->val;
          const int oi = o->idx;
          if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; cpos = o->pos; }
          if (p.n >= q * slice && p.n < q * slice + slice) s_wnew = o->wnew;
        }
        *ticket = 0;                     // ready for the next step (stream order)
      }
    }
  }
  __syncthreads();
  if (!s_last) return;
  if (tid == 0) {
    if (idx < 0 || idx > p.cap) { atomicExch(p.status, DEV_ERR_BAD_VICTIM); idx = p.cap; cpos = pos_t; }
    s_victim = idx;
    if (idx < p.cap) {
      table[idx] = pos_t;
      if (up.h2o) acc[idx] = s_wnew;
    }
    if (p.evicted) p.evicted[(size_t)b * up.units + u] = cpos;   // the new token's own position if it dropped itself
  }
  __syncthreads();
  const int victim = s_victim;
  if (victim < p.cap) {
    constexpr int RB16 = D * (int)sizeof(T) / 16;
    for (int i = tid; i < kv_n * RB16; i += UNIT_THREADS) {
      const int kv = kv0 + i / RB16;
      const size_t dst = (((size_t)b * p.Hkv + kv) * p.cap + victim) * RB16 + i % RB16;
      const size_t src = ((size_t)b * p.Hkv + kv) * RB16 + i % RB16;
      static_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[src];
      static_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[src];
    }
  }
}

}  // namespace tova
