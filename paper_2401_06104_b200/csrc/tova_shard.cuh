// One layer's state sharded by KV head over several GPUs (sm_100a).
//
// Algorithm 1 averages the last query's attention weights over the heads of the
// layer: a sum over heads.  With the KV heads (and the query heads that read
// them) split over `world` ranks, every rank streams its own heads exactly as a
// single GPU does; what the ranks must exchange before the arg-min is only
// each rank's partial head sum of the soft-max weights, one fp32 vector of
// capacity+1 entries per sequence.  The step therefore comes in two kernels
// around that exchange:
//
//   tova_shard_scores_kernel   after the streaming kernel: the partial sum
//       sum_{h local} p[h][j] / H_total for every candidate j, written into slot
//       `rank` of the score table of EVERY rank - plain stores into peer memory
//       (NVLink) - followed by a system-wide fence and, from the last thread block
//       to finish, this step's epoch into flag `rank` of every rank;
//   tova_shard_commit_kernel   waits (bounded) until all ranks' flags carry the
//       epoch, adds the partial vectors in rank order - the same bits on every
//       rank, so every rank picks the same victim - takes the arg-min (lowest
//       slot on ties, the new token being slot `capacity`) and writes the new
//       token's rows into its own KV heads (Eq. 9, in place).
//
// No TMA multicast and no library kernel touches peer memory: the exchange is
// made of ordinary st.global and ld.acquire.sys instructions.  When the caller
// prefers a library all-reduce (NCCL) it passes world = 1 tables and reduces
// the one vector itself between the two kernels.
#pragma once

#include "tova_kernels.cuh"

namespace tova {

constexpr int SHARD_MAX_WORLD = 8;
constexpr int SHARD_THREADS = 256;
constexpr int DEV_ERR_PEER_TIMEOUT = 3;   // a rank's partial sums did not arrive within the wait limit

struct ShardParams {
  float* parts[SHARD_MAX_WORLD];     // rank r's score table [2][tables][B][ld] (the halves alternate step by step: a
                                     // rank may already publish step t+1 while a slower one still adds up step t);
                                     // entry [rank] = this rank's own.  [B][ld] when the caller reduces
  int32_t* flags[SHARD_MAX_WORLD];   // rank r's flags [world]
  int32_t rank, world;               // this rank, number of ranks
  int32_t tables;                    // partial vectors to add in the commit kernel: world, or 1 when the caller reduces
  int32_t h_total;                   // query heads of the whole layer
  int32_t* epoch;                    // [1] local: steps exchanged so far
  int32_t* ticket;                   // [1] local: thread blocks of the scores kernel that have stored their part
};

__device__ __forceinline__ int32_t ld_acquire_sys(const int32_t* p) {
  int32_t v;
  asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
constexpr unsigned long long SHARD_WAIT_NS = 1000000000ull;   // how long a rank waits for its peers' parts

__device__ __forceinline__ void st_release_sys(int32_t* p, int32_t v) {
  asm volatile("st.release.sys.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// grid = (nx, B), block = SHARD_THREADS; dynamic shared memory: one float per local head.
// CTA x covers candidates [x*cand_per_cta, +cand_per_cta) of sequence b.
__global__ void __launch_bounds__(SHARD_THREADS) tova_shard_scores_kernel(const StepParams p, const ShardParams sp) {
  extern __shared__ __align__(16) float ssm[];
  float* hc = ssm;                                  // [H] -max2 - log2(sum * H_total)
  const int x = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NW = SHARD_THREADS / 32;
  if (p.fuse_out) {
    for (int h = tid; h < p.H; h += SHARD_THREADS) {
      const float2 e = p.head_ml[(size_t)b * p.H + h];
      hc[h] = -e.x - __log2f(e.y * (float)sp.h_total);
    }
  } else {
    const int np = p.n_chunks + 1;
    for (int h = warp; h < p.H; h += NW) {
      const float2* ml = p.part_ml + ((size_t)b * p.H + h) * p.pc;
      float M = -INFINITY;
      for (int i = lane; i < np; i += 32) M = fmaxf(M, ml[i].x);
      M = warp_max(M);
      float L = 0.f;
      for (int i = lane; i < np; i += 32) L = fmaf(ml[i].y, exp2_diff(ml[i].x, M), L);
      L = warp_sum(L);
      if (lane == 0) hc[h] = -M - __log2f(L * (float)sp.h_total);
    }
  }
  __syncthreads();
  const int j_begin = x * p.cand_per_cta, j_end = min(j_begin + p.cand_per_cta, p.n + 1);
  const float* lg = p.logits + (size_t)b * p.H * p.ld;
  const int e_next = (sp.tables > 1) ? *sp.epoch + 1 : 0;      // this step's epoch (written back by the last block only)
  const size_t slot = (((size_t)(e_next & 1) * sp.tables + (sp.tables > 1 ? sp.rank : 0)) * p.B + b) * p.ld;
  for (int j = j_begin + tid; j < j_end; j += SHARD_THREADS) {
    float a = 0.f;
    for (int h = 0; h < p.H; ++h) a += exp2f(lg[(size_t)h * p.ld + j] + hc[h]);
    if (sp.tables > 1) {
      for (int r = 0; r < sp.world; ++r) sp.parts[r][slot + j] = a;     // into every rank's table (peer stores)
    } else {
      sp.parts[sp.rank][slot + j] = a;                                    // the caller reduces this vector itself
    }
  }
  if (sp.tables > 1) {
    // Publish: all of this block's stores are ordered before its ticket; the block that takes the last ticket
    // tells every rank that this rank's part of the step is complete.
    __threadfence_system();
    __syncthreads();
    if (tid == 0) {
      const int total = gridDim.x * gridDim.y;
      if (atomicAdd(sp.ticket, 1) == total - 1) {
        *sp.ticket = 0;
        const int e = e_next;              // the commit kernel (later in the stream) reads it back
        *sp.epoch = e;
        __threadfence_system();
        for (int r = 0; r < sp.world; ++r) st_release_sys(sp.flags[r] + sp.rank, e);
      }
    }
  }
}

// grid = (B), block = SHARD_THREADS.  Adds the ranks' partial vectors in rank order, picks the victim, inserts.
template <typename T, int D>
__global__ void __launch_bounds__(SHARD_THREADS) tova_shard_commit_kernel(const StepParams p, const ShardParams sp) {
  constexpr int NW = SHARD_THREADS / 32;
  constexpr int RB16 = D * (int)sizeof(T) / 16;
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  __shared__ float red_v[NW];
  __shared__ int red_i[NW];
  __shared__ int red_p[NW];
  __shared__ int s_victim;
  __shared__ int s_ok;
  const int pos_t = *p.cur_pos;
  const int row_words = p.Hkv * RB16;

  auto insert_row = [&](int slot) {
    for (int i = tid; i < row_words; i += SHARD_THREADS) {
      const size_t dst = (((size_t)b * p.Hkv + i / RB16) * p.cap + slot) * RB16 + i % RB16;
      static_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[(size_t)b * row_words + i];
      static_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[(size_t)b * row_words + i];
    }
  };
  if (!p.do_evict) {                 // g(t) = min(t, k) not reached: nothing was exchanged, the token takes the next row
    insert_row(p.n);
    if (tid == 0) {
      p.pos[(size_t)b * p.cap + p.n] = pos_t;
      p.len[b] = p.n + 1;
      if (p.last_slot) p.last_slot[b] = p.n;
      if (p.evicted) p.evicted[b] = -1;
    }
    return;
  }
  // ---- wait for every rank's part of this step (bounded) -----------------------------------------------
  const int e = *sp.epoch;           // set by this rank's scores kernel of the same step
  if (tid == 0) s_ok = 1;
  __syncthreads();
  if (sp.tables > 1 && tid < sp.world) {        // thread r watches rank r's flag, for about a second at most
    const unsigned long long t0 = global_ns();
    bool seen = false;
    while (!(seen = ld_acquire_sys(sp.flags[sp.rank] + tid) >= e) && global_ns() - t0 < SHARD_WAIT_NS) {}
    if (!seen) s_ok = 0;
  }
  __syncthreads();
  if (!s_ok) {                       // report and leave the state as it is: the context stays usable
    if (tid == 0) atomicExch(p.status, DEV_ERR_PEER_TIMEOUT);
    return;
  }
  // ---- the layer's head-averaged weights: the parts in rank order; lowest (value, slot) ---------------------
  const float* base = sp.parts[sp.rank] + ((size_t)(sp.tables > 1 ? (e & 1) : 0) * sp.tables * p.B + b) * p.ld;
  const size_t tstride = (size_t)p.B * p.ld;
  float val = INFINITY;
  int idx = 0x7fffffff, cpos = pos_t;
  for (int j = tid; j <= p.n; j += SHARD_THREADS) {
    float a = 0.f;
    for (int r = 0; r < sp.tables; ++r) a += __ldcg(base + r * tstride + j);
    const int pj = (j < p.cap) ? p.pos[(size_t)b * p.cap + j] : pos_t;
    if (pj < p.keep_first) a = INFINITY;           // one of the first i token states: never dropped
    if (a < val) { val = a; idx = j; cpos = pj; }
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    const int op = __shfl_xor_sync(0xffffffffu, cpos, o);
    if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; cpos = op; }
  }
  if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; red_p[warp] = cpos; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < NW; ++w)
      if (red_v[w] < val || (red_v[w] == val && red_i[w] < idx)) { val = red_v[w]; idx = red_i[w]; cpos = red_p[w]; }
    if (idx < 0 || idx > p.cap) { atomicExch(p.status, DEV_ERR_BAD_VICTIM); idx = p.cap; cpos = pos_t; }
    s_victim = idx;
    if (idx < p.cap) p.pos[(size_t)b * p.cap + idx] = pos_t;
    if (p.last_slot) p.last_slot[b] = (idx < p.cap) ? idx : -1;
    if (p.evicted) p.evicted[b] = cpos;
  }
  __syncthreads();
  if (s_victim < p.cap) insert_row(s_victim);
}

}  // namespace tova
