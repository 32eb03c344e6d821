// Prompt tokens beyond the capacity, many per launch (sm_100a).
//
// Once the state is full every prompt token drops a row (Algorithm 1), and the
// row it drops changes what the next token attends to: taken literally that is
// one dependent decode step per token.  The paper's language-modelling runs
// avoid this by editing the attention mask of a whole chunk of tokens according
// to the attention weights of the layer (appendix "Experimental Details"); the
// same idea, made exact, drives this file.  For a chunk of up to 64 tokens that
// meets a full state:
//
//   stage     the chunk's keys and values are copied next to the state
//             (tova_chunk_stage_kernel) so that tiled copies can reach them;
//   logits    ONE dense pass computes the scaled logits of all the chunk's
//             queries against every row they could possibly attend to - the k
//             rows of the state as the chunk found it, and the chunk's own
//             earlier tokens - plus each query's row maximum R and the sum T of
//             exp2(logit - R) over all those columns (tova_chunk_attn_kernel,
//             MODE 0; warp-level bf16 MMAs, as in the bulk fill);
//   resolve   a cluster of thread blocks per sequence that share out the slots,
//             with the logits staged in shared memory
//             (tova_chunk_resolve_cluster1_kernel, one cluster barrier per token;
//             tova_chunk_resolve_cluster_kernel, two) - or one block per sequence
//             reading global memory (tova_chunk_resolve_kernel) - replays the
//             chunk's deletions in order from those logits alone: for token i it
//             removes the rows dropped by tokens < i from the normaliser
//             (L = T - their terms), scores the k+1 live candidates
//             by the head-averaged soft-max weight (Eq. 4, Algorithm 1), takes
//             the arg-min - lowest slot on ties, the token itself being slot k -
//             records the dropped position and lets the token take the slot.
//             No key or value is touched: per token the work is H*(k+1) exp2;
//   outputs   a second dense pass forms Eq. 7 for every query with the weights
//             masked to the rows alive at ITS step and normalised by ITS L
//             (tova_chunk_attn_kernel, MODE 1);
//   scatter   the surviving tokens' rows go to the slots they won
//             (tova_chunk_scatter_kernel).
//
// The result is what token-by-token steps give: the same candidates, weights
// and arg-min per token, up to floating-point summation order (near-ties closer
// than rounding can fall either way, as between any two implementations).
#pragma once

#include <cooperative_groups.h>
#include <cuda.h>

#include "tova_fill.cuh"

namespace tova {

constexpr int CHUNK_TOKENS = 64;        // tokens per chunk = query rows of one attention CTA = rows of one staging tile
constexpr int CHUNK_RESOLVE_THREADS = 1024;

struct ChunkParams {
  // state
  unsigned char* K;        // [B,Hkv,cap,D]
  unsigned char* V;
  int32_t* pos;            // [B,cap]
  int32_t* cur_pos;        // [1]
  int32_t* last_slot;      // [B]
  int32_t* status;         // [1]
  // the chunk's tokens
  const void* q;           // [C,B,H,D]
  const void* k_new;       // [C,B,Hkv,D]
  const void* v_new;
  float* out;              // [C,B,H,D] or null
  int32_t* evicted;        // [C,B] or null
  // workspace
  unsigned char* Kst;      // [B,Hkv,64,D] the chunk's keys
  unsigned char* Vst;
  float* lg;               // [B,64,H,ldc] base-2 logits of query i, head h: columns 0..cap-1 = state rows,
                           // capA+j = chunk token j (capA = cap rounded up to 4: 16-byte aligned blocks)
  float2* rt;              // [B,H,64] (row maximum R, sum T of exp2(logit - R) over all columns a query can see)
  float2* ml;              // [B,H,64] (R, sum L over the candidates alive at the query's step)
  int32_t* death;          // [B,ldc] step at which a column's token is dropped (it is still attended at that step)
  int32_t* slot_token;     // [B,cap] chunk token that ends up in a slot, -1: the slot keeps its row
  int32_t* first;          // [1] position of the chunk's first token
  int B, H, Hkv, G, cap, capA, ldc;
  int C;                   // tokens in this chunk (1..64)
  int first_pos;           // position of the chunk's first token, or < 0: current position + 1
  int keep_first;          // rows holding positions 0..keep_first-1 are never dropped
  int window;              // 1: the Window policy - the row holding the earliest droppable position goes
  float scale2;
};

constexpr int32_t CHUNK_ALIVE = 0x7fffffff;

// 2^x by the special-function unit alone; results below the smallest normal number become zero.
__device__ __forceinline__ float exp2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The chunk's keys/values into the staging tiles (rows past the chunk are zeroed: they are read with weight zero),
// every column's death step reset, the first position fixed for the later kernels.
template <int D>
__global__ void tova_chunk_stage_kernel(const ChunkParams p) {
  constexpr int CH = D * 2 / 16;
  const size_t total = (size_t)p.B * p.Hkv * CHUNK_TOKENS * CH;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int ch = (int)(i % CH);
    const size_t row = i / CH;                         // (b, kvh, t)
    const int t = (int)(row % CHUNK_TOKENS);
    const size_t bk = row / CHUNK_TOKENS;              // b * Hkv + kvh
    uint4 kq = make_uint4(0u, 0u, 0u, 0u), vq = kq;
    if (t < p.C) {
      const size_t src = ((size_t)t * p.B * p.Hkv + bk) * CH + ch;
      kq = static_cast<const uint4*>(p.k_new)[src];
      vq = static_cast<const uint4*>(p.v_new)[src];
    }
    reinterpret_cast<uint4*>(p.Kst)[i] = kq;
    reinterpret_cast<uint4*>(p.Vst)[i] = vq;
  }
  const size_t nd = (size_t)p.B * p.ldc;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nd; i += (size_t)gridDim.x * blockDim.x)
    p.death[i] = CHUNK_ALIVE;
  if (blockIdx.x == 0 && threadIdx.x == 0) *p.first = (p.first_pos < 0) ? *p.cur_pos + 1 : p.first_pos;
}

// MODE 0: logits of the chunk's queries against the state and the chunk, row maxima and row sums.
// MODE 1: attention outputs with the weights masked per query step and normalised by the resolved sums.
// grid = (H, B), block = 128: warp w owns queries 16w..16w+15 of the chunk.  Tiles of 64 rows: the state's
// (through map_k / map_v), then the chunk's own (map_ks / map_vs).  Dynamic shared memory as the bulk fill's.
template <int D, int MODE>
__global__ void __launch_bounds__(FILL_THREADS, 3) tova_chunk_attn_kernel(const ChunkParams p,
                                                                       const __grid_constant__ CUtensorMap map_k,
                                                                       const __grid_constant__ CUtensorMap map_v,
                                                                       const __grid_constant__ CUtensorMap map_ks,
                                                                       const __grid_constant__ CUtensorMap map_vs) {
  constexpr int TILE_BYTES = FILL_K_ROWS * D * 2;
  constexpr int BOXES = D / 64;
  constexpr int KS = D / 16;
  constexpr int ND = D / 8;

  extern __shared__ unsigned char chunk_smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(chunk_smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* kv_s = smem;                              // stage s: K at 2s, V at 2s+1
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ int32_t dth[2][FILL_K_ROWS];                  // MODE 1: death step of the tile's columns

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y;
  const int kvh = h / p.G;
  const int head_row0 = (b * p.Hkv + kvh) * p.cap;         // first row of this head in the [B*Hkv*cap, D] view
  const int stage_row0 = (b * p.Hkv + kvh) * CHUNK_TOKENS; // ... in the [B*Hkv*64, D] view of the staging tiles
  const int n_state = (p.cap + FILL_K_ROWS - 1) / FILL_K_ROWS;
  const int n_tiles = n_state + 1;

  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue = [&](int i) {
    uint64_t* bar = &bars[i & 1];
    unsigned char* kd = kv_s + (size_t)(2 * (i & 1)) * TILE_BYTES;
    unsigned char* vd = kd + TILE_BYTES;
    mbar_expect_tx(bar, (MODE == 1 ? 2u : 1u) * TILE_BYTES);
    const bool st = i < n_state;
    const int y = st ? head_row0 + i * FILL_K_ROWS : stage_row0;
#pragma unroll
    for (int bx = 0; bx < BOXES; ++bx) {
      tma_load_2d_keep(kd + bx * (FILL_K_ROWS * 128), st ? &map_k : &map_ks, bx * 64, y, bar);
      if (MODE == 1) tma_load_2d_keep(vd + bx * (FILL_K_ROWS * 128), st ? &map_v : &map_vs, bx * 64, y, bar);
    }
  };
  if (tid == 0) issue(0);

  // A fragments of this warp's 16 query rows, straight from global memory; rows past the chunk repeat its last token.
  const int row_lo = warp * 16 + (lane >> 2);
  const int qa_i = min(row_lo, p.C - 1), qb_i = min(row_lo + 8, p.C - 1);
  uint32_t qa[KS][4];
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q);
    const uint32_t* qra = reinterpret_cast<const uint32_t*>(qg + (((size_t)qa_i * p.B + b) * p.H + h) * D) + (lane & 3);
    const uint32_t* qrb = reinterpret_cast<const uint32_t*>(qg + (((size_t)qb_i * p.B + b) * p.H + h) * D) + (lane & 3);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = __ldg(qra + ks * 8);
      qa[ks][1] = __ldg(qrb + ks * 8);
      qa[ks][2] = __ldg(qra + ks * 8 + 4);
      qa[ks][3] = __ldg(qrb + ks * 8 + 4);
    }
  }
  const size_t bh = (size_t)b * p.H + h;
  float* lg0 = p.lg + (((size_t)b * CHUNK_TOKENS + qa_i) * p.H + h) * p.ldc;   // this lane's two logit rows
  float* lg1 = p.lg + (((size_t)b * CHUNK_TOKENS + qb_i) * p.H + h) * p.ldc;
  const bool real0 = row_lo < p.C, real1 = row_lo + 8 < p.C;

  float o[ND][4];
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float R0 = 0.f, R1 = 0.f, iL0 = 0.f, iL1 = 0.f;
  if (MODE == 1) {
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;
    const float2 a = p.ml[bh * CHUNK_TOKENS + qa_i], c = p.ml[bh * CHUNK_TOKENS + qb_i];
    R0 = a.x; iL0 = 1.f / a.y;
    R1 = c.x; iL1 = 1.f / c.y;
  }
  const int32_t* death = p.death + (size_t)b * p.ldc;
  bool ok = true;

  for (int i = 0; i < n_tiles; ++i) {
    if (tid == 0 && i + 1 < n_tiles) issue(i + 1);
    const bool st = i < n_state;
    const int c0 = st ? i * FILL_K_ROWS : p.capA;           // column of the tile's first row
    if (MODE == 1 && tid < FILL_K_ROWS) {
      const int c = c0 + tid;
      dth[i & 1][tid] = (c < p.ldc) ? death[c] : -1;
    }
    ok = warp_wait(&bars[i & 1], (uint32_t)((i >> 1) & 1)) && ok;
    if (MODE == 1) __syncthreads();
    const uint32_t kt = smem_addr(kv_s + (size_t)(2 * (i & 1)) * TILE_BYTES);
    const uint32_t vt = kt + TILE_BYTES;

    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int kr = nt * 8 + (lane & 7);
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        uint32_t kb[4];
        ldmatrix_x4(kb, kt + fill_swz(kr, 2 * ks + (lane >> 3)));
        mma_bf16(s[nt], qa[ks], kb[0], kb[1]);
        mma_bf16(s[nt], qa[ks + 1], kb[2], kb[3]);
      }
    }

    // Which columns a query may see: every row of the state (tile rows past the capacity belong to the next head),
    // and the chunk's tokens up to itself.
    const int lim = st ? p.cap - c0 : 0;                    // state tile: rows < lim are this head's
    if (MODE == 0) {
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int r = nt * 8 + 2 * (lane & 3);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool v0 = st ? (r + e < lim) : (r + e <= qa_i);
          const bool v1 = st ? (r + e < lim) : (r + e <= qb_i);
          const float a = v0 ? s[nt][e] * p.scale2 : -INFINITY, c = v1 ? s[nt][2 + e] * p.scale2 : -INFINITY;
          s[nt][e] = a;
          s[nt][2 + e] = c;
          mx0 = fmaxf(mx0, a);
          mx1 = fmaxf(mx1, c);
        }
        // keep the logits: two neighbouring columns per store (columns a query cannot see are never read back)
        const int c = c0 + r;                       // even: 8-byte aligned pairs
        const bool k0 = !st || r < lim, k1 = !st || r + 1 < lim;
        if (k0 && k1) {
          if (real0) *reinterpret_cast<float2*>(lg0 + c) = make_float2(s[nt][0], s[nt][1]);
          if (real1) *reinterpret_cast<float2*>(lg1 + c) = make_float2(s[nt][2], s[nt][3]);
        } else {
          if (k0 && real0) lg0[c] = s[nt][0];
          if (k0 && real1) lg1[c] = s[nt][2];
          if (k1 && real0) lg0[c + 1] = s[nt][1];
          if (k1 && real1) lg1[c + 1] = s[nt][3];
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);   // finite from tile 0 on: the state is full
      l_run[0] *= exp2_diff(m_run[0], mn0);
      l_run[1] *= exp2_diff(m_run[1], mn1);
      m_run[0] = mn0;
      m_run[1] = mn1;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        l_run[0] += exp2f(s[nt][0] - mn0) + exp2f(s[nt][1] - mn0);
        l_run[1] += exp2f(s[nt][2] - mn1) + exp2f(s[nt][3] - mn1);
      }
    } else {
      // weights of the rows alive at the query's step: born no later (chunk tokens), dropped no earlier
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int nt = 2 * kk + half;
          const int r = nt * 8 + 2 * (lane & 3);
          float e4[4];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int dd = dth[i & 1][r + e];
            const bool v0 = (st ? (r + e < lim) : (r + e <= qa_i)) && dd >= qa_i;
            const bool v1 = (st ? (r + e < lim) : (r + e <= qb_i)) && dd >= qb_i;
            e4[e] = v0 ? exp2f(s[nt][e] * p.scale2 - R0) : 0.f;
            e4[2 + e] = v1 ? exp2f(s[nt][2 + e] * p.scale2 - R1) : 0.f;
          }
          split_hi_lo(e4[0], e4[1], ph[2 * half], pl[2 * half]);
          split_hi_lo(e4[2], e4[3], ph[2 * half + 1], pl[2 * half + 1]);
        }
        const int vr = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int nd = 0; nd < ND; nd += 2) {
          uint32_t vb[4];
          ldmatrix_x4_trans(vb, vt + fill_swz(vr, nd + (lane >> 4)));
          mma_bf16(o[nd], ph, vb[0], vb[1]);
          mma_bf16(o[nd], pl, vb[0], vb[1]);
          mma_bf16(o[nd + 1], ph, vb[2], vb[3]);
          mma_bf16(o[nd + 1], pl, vb[2], vb[3]);
        }
      }
    }
    fence_proxy_async_smem();
    __syncthreads();
  }

  if (!ok) {
    if (tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    return;
  }

  if (MODE == 0) {
    float l0 = l_run[0], l1 = l_run[1];
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    if ((lane & 3) == 0) {
      if (real0) p.rt[bh * CHUNK_TOKENS + row_lo] = make_float2(m_run[0], l0);
      if (real1) p.rt[bh * CHUNK_TOKENS + row_lo + 8] = make_float2(m_run[1], l1);
    }
  } else {
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) {
      const int d = nd * 8 + 2 * (lane & 3);
      if (real0)
        *reinterpret_cast<float2*>(p.out + (((size_t)row_lo * p.B + b) * p.H + h) * D + d) =
            make_float2(o[nd][0] * iL0, o[nd][1] * iL0);
      if (real1)
        *reinterpret_cast<float2*>(p.out + (((size_t)(row_lo + 8) * p.B + b) * p.H + h) * D + d) =
            make_float2(o[nd][2] * iL1, o[nd][3] * iL1);
    }
  }
}

// The chunk's deletions, in order, from the logits alone.  grid = (B), block = CHUNK_RESOLVE_THREADS.
// Dynamic shared memory: occupant column and position of every slot (2 x cap ints), per-head constants (H floats).
__global__ void __launch_bounds__(CHUNK_RESOLVE_THREADS) tova_chunk_resolve_kernel(const ChunkParams p) {
  constexpr int NT = CHUNK_RESOLVE_THREADS, NW = NT / 32;
  extern __shared__ __align__(16) int32_t rsm[];
  int32_t* occ = rsm;                    // [cap] column whose token sits in the slot
  int32_t* posv = occ + p.cap;           // [cap] position that token holds
  float* hc = reinterpret_cast<float*>(posv + p.cap);   // [H] -R - log2(L * H) of the current query
  __shared__ int32_t dead[CHUNK_TOKENS]; // columns dropped so far in this chunk
  __shared__ float red_v[NW];
  __shared__ int red_i[NW];
  __shared__ int s_ndead;

  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int first = *p.first;
  for (int s = tid; s < p.cap; s += NT) {
    occ[s] = s;
    posv[s] = p.pos[(size_t)b * p.cap + s];
  }
  if (tid == 0) s_ndead = 0;
  __syncthreads();

  const float* lgb = p.lg + (size_t)b * CHUNK_TOKENS * p.H * p.ldc;
  const size_t hstride = (size_t)p.ldc;                 // between heads
  for (int i = 0; i < p.C; ++i) {
    const int pos_i = first + i;
    const float* row = lgb + (size_t)i * p.H * p.ldc;    // head 0's logits of query i
    const int ndead = s_ndead;
    // ---- each head's normaliser over the rows alive now: the sum over all columns minus the dropped ones ----
    for (int h = warp; h < p.H; h += NW) {
      const float2 rt = p.rt[((size_t)b * p.H + h) * CHUNK_TOKENS + i];
      float gone = 0.f;
      for (int d = lane; d < ndead; d += 32) gone += exp2f(row[h * hstride + dead[d]] - rt.x);
      gone = warp_sum(gone);
      if (lane == 0) {
        const float L = rt.y - gone;
        hc[h] = -rt.x - __log2f(L * (float)p.H);
        p.ml[((size_t)b * p.H + h) * CHUNK_TOKENS + i] = make_float2(rt.x, L);
      }
    }
    __syncthreads();
    // ---- head-averaged weight of the k+1 candidates (Algorithm 1), lowest first -------------------------
    float val = INFINITY;
    int idx = 0x7fffffff;
    for (int s = tid; s <= p.cap; s += NT) {
      const int c = (s < p.cap) ? occ[s] : p.capA + i;
      const int pj = (s < p.cap) ? posv[s] : pos_i;
      const float* col = row + c;
      float a = 0.f;
#pragma unroll 8
      for (int h = 0; h < p.H; ++h) a += exp2f(col[h * hstride] + hc[h]);
      if (p.window) a = (float)(pj - pos_i);             // Window: the earliest position goes (ages are below 2^24: exact)
      if (pj < p.keep_first) a = INFINITY;               // one of the first i token states: never dropped
      if (a < val) { val = a; idx = s; }                 // s ascends: strict < keeps the lowest slot
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, val, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; }
    }
    if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < NW; ++w)
        if (red_v[w] < val || (red_v[w] == val && red_i[w] < idx)) { val = red_v[w]; idx = red_i[w]; }
      if (idx < 0 || idx > p.cap) { atomicExch(p.status, DEV_ERR_BAD_VICTIM); idx = p.cap; }
      int gone_col, gone_pos;
      if (idx < p.cap) {                                 // the token takes the dropped row's slot (Eq. 9, in place)
        gone_col = occ[idx];
        gone_pos = posv[idx];
        occ[idx] = p.capA + i;
        posv[idx] = pos_i;
      } else {                                           // the token itself had the lowest weight
        gone_col = p.capA + i;
        gone_pos = pos_i;
      }
      p.death[(size_t)b * p.ldc + gone_col] = i;
      dead[ndead] = gone_col;
      s_ndead = ndead + 1;
      if (p.evicted) p.evicted[(size_t)i * p.B + b] = gone_pos;
    }
    __syncthreads();
  }
  for (int s = tid; s < p.cap; s += NT) {
    p.pos[(size_t)b * p.cap + s] = posv[s];
    p.slot_token[(size_t)b * p.cap + s] = (occ[s] >= p.capA) ? occ[s] - p.capA : -1;
  }
}

// The same replay with the candidates of a sequence spread over a thread-block cluster and the logits staged in
// shared memory ahead of time.  grid = (NC, B), cluster (NC,1,1), block = 256.  CTA r owns slots [r*S, r*S+S)
// (S a multiple of 4); CTA 0 also owns the new token (candidate `capacity`).  Per token every CTA needs, of each
// head's logit row, its own S state columns and the 64 chunk columns (a slot's occupant may by now be a chunk
// token): 2*H bulk copies into one of `nstage` buffers, requested nstage tokens ahead - what a token reads
// does not depend on earlier deletions, only which of the staged columns it uses does.  Per token:
//   A. every warp takes heads, its lanes the CTA's candidates: e = exp2(logit - R) in place, the head's partial sum
//      goes to every CTA of the cluster (distributed shared memory);           cluster barrier
//   B. L_h = the partial sums in rank order; every thread scores a candidate: sum_h e[h] / (L_h * H); block arg-min;
//      the CTA's best (value, slot) goes to every CTA;                          cluster barrier
//   C. every CTA takes the same arg-min over the NC entries (lowest slot on ties); the owner of the slot
//      replaces its occupant; the buffer is handed back to the copy engine for token i + nstage.
// All waits on copies are bounded; a wait that runs out sets the status word and the kernel carries on through
// its barriers (peers must not be left waiting).
constexpr int CHUNK_CLUSTER_THREADS_MAX = 1024;   // block size: about one thread per candidate of the CTA, 256..1024
constexpr int CHUNK_CLUSTER_MAX = 8;
constexpr int CHUNK_STAGES_MAX = 4;

__host__ __device__ inline size_t chunk_cluster_smem(int H, int S, int nstage) {
  return sizeof(float) * ((size_t)nstage * H * (S + CHUNK_TOKENS) + (size_t)CHUNK_TOKENS * H +
                          2 * (size_t)CHUNK_CLUSTER_MAX * H + H) + sizeof(int32_t) * 2 * (size_t)S + 64;
}

__global__ void __launch_bounds__(CHUNK_CLUSTER_THREADS_MAX) tova_chunk_resolve_cluster_kernel(const ChunkParams p,
                                                                                           const int S, const int nstage) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  constexpr int NWM = CHUNK_CLUSTER_THREADS_MAX / 32, NCM = CHUNK_CLUSTER_MAX;
  const int NT = (int)blockDim.x, NW = NT / 32;
  const int NC = (int)cl.num_blocks(), r = (int)cl.block_rank();
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = p.H, SW = S + CHUNK_TOKENS;

  extern __shared__ __align__(16) float csm2[];
  float* stage = csm2;                                        // [nstage][H][SW]
  float* Rs = stage + (size_t)nstage * H * SW;               // [64][H] row maxima of the chunk's queries
  float* part = Rs + (size_t)CHUNK_TOKENS * H;               // [2][NCM][H] partial sums of every CTA, double-buffered
  float* invLH = part + 2 * (size_t)NCM * H;                 // [H] 1 / (L_h * H)
  int32_t* occl = reinterpret_cast<int32_t*>(invLH + H);     // [S] staged column holding the slot's occupant
  int32_t* posv = occl + S;                                  // [S] position it holds
  __shared__ __align__(8) uint64_t full[CHUNK_STAGES_MAX];
  __shared__ float2 best[2][NCM];                            // (value, slot) of every CTA, double-buffered
  __shared__ float red_v[NWM];
  __shared__ int red_i[NWM];

  const int s_begin = r * S;
  const int n_loc = max(0, min(S, p.cap - s_begin));          // slots this CTA really owns
  const int n_cand = n_loc + (r == 0 ? 1 : 0);                // plus the new token
  const int first = *p.first;
  const float* lgb = p.lg + (size_t)b * CHUNK_TOKENS * H * p.ldc;

  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) mbar_init(&full[s], 1);
    mbar_fence_init();
  }
  for (int t = tid; t < S; t += NT) {
    occl[t] = t;
    posv[t] = (t < n_loc) ? p.pos[(size_t)b * p.cap + s_begin + t] : 0;
  }
  for (int t = tid; t < CHUNK_TOKENS * H; t += NT) {
    const int i = t / H, h = t % H;
    Rs[t] = (i < p.C) ? p.rt[((size_t)b * H + h) * CHUNK_TOKENS + i].x : 0.f;
  }
  __syncthreads();
  // logits of token i into buffer i % nstage (warp 0): per head the CTA's state columns and the chunk's columns
  auto request = [&](int i) {
    uint64_t* bar = &full[i % nstage];
    float* dst = stage + (size_t)(i % nstage) * H * SW;
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)H * (uint32_t)SW * 4u);
    __syncwarp();
    const float* src = lgb + (size_t)i * H * p.ldc;
    for (int h = lane; h < H; h += 32) {
      bulk_g2s(dst + (size_t)h * SW, src + (size_t)h * p.ldc + s_begin, (uint32_t)S * 4u, bar);
      bulk_g2s(dst + (size_t)h * SW + S, src + (size_t)h * p.ldc + p.capA, (uint32_t)CHUNK_TOKENS * 4u, bar);
    }
  };
  if (warp == 0)
    for (int i = 0; i < min(nstage, p.C); ++i) request(i);
  cl.sync();                                                  // every CTA of the cluster runs: its shared memory may be written

  bool ok = true;
  for (int i = 0; i < p.C; ++i) {
    const int pos_i = first + i;
    const int par = i & 1;
    float* st = stage + (size_t)(i % nstage) * H * SW;
    ok = warp_wait(&full[i % nstage], (uint32_t)((i / nstage) & 1)) && ok;
    // ---- A: un-normalised weights in place, per-head partial sums to every CTA ---------------------
    for (int h = warp; h < H; h += NW) {
      const float R = Rs[i * H + h];
      float* row = st + (size_t)h * SW;
      float sum = 0.f;
      int t = lane;
      for (; t + 96 < n_cand; t += 128) {                 // four independent candidates in flight per lane
        int c[4];
        float e[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) c[u] = (t + 32 * u < n_loc) ? occl[t + 32 * u] : S + i;
#pragma unroll
        for (int u = 0; u < 4; ++u) e[u] = exp2f(row[c[u]] - R);
#pragma unroll
        for (int u = 0; u < 4; ++u) { row[c[u]] = e[u]; sum += e[u]; }
      }
      for (; t < n_cand; t += 32) {
        const int c = (t < n_loc) ? occl[t] : S + i;
        const float e = exp2f(row[c] - R);
        row[c] = e;
        sum += e;
      }
      sum = warp_sum(sum);
      if (lane < NC) *cl.map_shared_rank(&part[((size_t)par * NCM + r) * H + h], lane) = sum;
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    for (int h = tid; h < H; h += NT) {
      float L = 0.f;
      for (int rr = 0; rr < NC; ++rr) L += part[((size_t)par * NCM + rr) * H + h];
      invLH[h] = 1.f / (L * (float)H);
      if (r == 0) p.ml[((size_t)b * H + h) * CHUNK_TOKENS + i] = make_float2(Rs[i * H + h], L);
    }
    __syncthreads();
    // ---- B: head-averaged weight of this CTA's candidates, lowest (value, slot) ----------------------
    float val = INFINITY;
    int idx = 0x7fffffff;
    for (int t = tid; t < n_cand; t += NT) {
      const int c = (t < n_loc) ? occl[t] : S + i;
      const int pj = (t < n_loc) ? posv[t] : pos_i;
      const float* col = st + c;
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;       // fixed order: heads h = 0,4,8,.. / 1,5,.. / 2,6,.. / 3,7,..
      int h = 0;
      for (; h + 3 < H; h += 4) {
        a0 = fmaf(col[(size_t)h * SW], invLH[h], a0);
        a1 = fmaf(col[(size_t)(h + 1) * SW], invLH[h + 1], a1);
        a2 = fmaf(col[(size_t)(h + 2) * SW], invLH[h + 2], a2);
        a3 = fmaf(col[(size_t)(h + 3) * SW], invLH[h + 3], a3);
      }
      for (; h < H; ++h) a0 = fmaf(col[(size_t)h * SW], invLH[h], a0);
      float a = (a0 + a1) + (a2 + a3);
      if (p.window) a = (float)(pj - pos_i);             // Window: the earliest position goes
      if (pj < p.keep_first) a = INFINITY;
      const int g = (t < n_loc) ? s_begin + t : p.cap;
      if (a < val) { val = a; idx = g; }               // t ascends and with it the slot: strict < keeps the lowest
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, val, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; }
    }
    if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; }
    __syncthreads();
    if (warp == 0) {
      val = (lane < NW) ? red_v[lane] : INFINITY;
      idx = (lane < NW) ? red_i[lane] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, val, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; }
      }
      if (lane < NC) *cl.map_shared_rank(&best[par][r], lane) = make_float2(val, __int_as_float(idx));
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    // ---- C: the same arg-min in every CTA; the slot's owner lets the token in ---------------------------------
    float bv = INFINITY;
    int bi = 0x7fffffff;
    for (int rr = 0; rr < NC; ++rr) {
      const float2 e = best[par][rr];
      const int ei = __float_as_int(e.y);
      if (e.x < bv || (e.x == bv && ei < bi)) { bv = e.x; bi = ei; }
    }
    if (bi < 0 || bi > p.cap) {                          // cannot happen with finite logits: report, drop the token
      if (tid == 0 && r == 0) atomicExch(p.status, DEV_ERR_BAD_VICTIM);
      bi = p.cap;
    }
    if (tid == 0) {
      if (bi < p.cap) {
        const int l = bi - s_begin;
        if (l >= 0 && l < n_loc) {                      // Eq. 9 in place: the token takes the dropped row's slot
          const int old = occl[l];
          p.death[(size_t)b * p.ldc + (old < S ? s_begin + old : p.capA + (old - S))] = i;
          if (p.evicted) p.evicted[(size_t)i * p.B + b] = posv[l];
          occl[l] = S + i;
          posv[l] = pos_i;
        }
      } else if (r == 0) {                               // the token itself had the lowest weight
        p.death[(size_t)b * p.ldc + p.capA + i] = i;
        if (p.evicted) p.evicted[(size_t)i * p.B + b] = pos_i;
      }
    }
    __syncthreads();                                     // the buffer has been read by everybody; occl is up to date
    if (warp == 0 && i + nstage < p.C) {
      fence_proxy_async_smem();
      request(i + nstage);
    }
  }
  if (!ok && tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
  for (int t = tid; t < n_loc; t += NT) {
    p.pos[(size_t)b * p.cap + s_begin + t] = posv[t];
    p.slot_token[(size_t)b * p.cap + s_begin + t] = (occl[t] >= S) ? occl[t] - S : -1;
  }
}

// The same replay with ONE cluster barrier per token (used where at least two tokens' logits fit in shared memory).
// The normaliser of a token needs no pass of its own: L = T - (terms of the columns dropped so far), T being the
// row sum over all columns that the logits pass left behind.  Every CTA keeps the list of the columns that died in
// ITS slots (CTA 0 also of the tokens that dropped themselves) and, while token i is being decided, adds up their
// terms for token i+1; the column that dies AT token i is not known before the barrier, so every CTA sends, with its
// candidate for the arg-min, that candidate's terms for token i+1.  After the barrier every CTA holds the same
// arg-min, the winner's terms and all partial corrections: L of token i+1 follows without another exchange, and the
// candidates are scored in a single pass (exp2 of logit - R - log2(L H), summed over the heads).
__host__ __device__ inline size_t chunk_cluster1_smem(int H, int S, int nstage) {
  return sizeof(float) * ((size_t)nstage * H * (S + CHUNK_TOKENS) + 2 * (size_t)CHUNK_TOKENS * H +
                          4 * (size_t)CHUNK_CLUSTER_MAX * H + 2 * (size_t)H) +
         sizeof(int32_t) * 2 * (size_t)S + 64;
}

__global__ void __launch_bounds__(CHUNK_CLUSTER_THREADS_MAX) tova_chunk_resolve_cluster1_kernel(const ChunkParams p,
                                                                                            const int S, const int nstage) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  constexpr int NWM = CHUNK_CLUSTER_THREADS_MAX / 32, NCM = CHUNK_CLUSTER_MAX;
  const int NT = (int)blockDim.x, NW = NT / 32;
  const int NC = (int)cl.num_blocks(), r = (int)cl.block_rank();
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = p.H, SW = S + CHUNK_TOKENS;

  extern __shared__ __align__(16) float csm3[];
  float* stage = csm3;                                        // [nstage][H][SW]
  float* Rs = stage + (size_t)nstage * H * SW;               // [64][H] row maxima of the chunk's queries
  float* Ts = Rs + (size_t)CHUNK_TOKENS * H;                 // [64][H] row sums over all columns
  float* xen = Ts + (size_t)CHUNK_TOKENS * H;                // [2][NCM][H] every CTA's candidate: its terms for the next token
  float* xco = xen + 2 * (size_t)NCM * H;                    // [2][NCM][H] every CTA's correction for the next token
  float* hc = xco + 2 * (size_t)NCM * H;                     // [H] -R - log2(L * H) of the current token
  float* s_co = hc + H;                                      // [H] this CTA's correction for the next token
  int32_t* occl = reinterpret_cast<int32_t*>(s_co + H);   // [S] staged column holding the slot's occupant
  int32_t* posv = occl + S;                                  // [S] position it holds
  __shared__ __align__(8) uint64_t full[CHUNK_STAGES_MAX];
  __shared__ float2 best[2][NCM];                            // (value, slot) of every CTA, double-buffered
  __shared__ float red_v[NWM];
  __shared__ int red_i[NWM], red_c[NWM];
  __shared__ int32_t dead[CHUNK_TOKENS];                     // staged columns that died in this CTA's care
  __shared__ int s_ndead;

  const int s_begin = r * S;
  const int n_loc = max(0, min(S, p.cap - s_begin));          // slots this CTA really owns
  const int n_cand = n_loc + (r == 0 ? 1 : 0);                // plus the new token
  const int first = *p.first;
  const float* lgb = p.lg + (size_t)b * CHUNK_TOKENS * H * p.ldc;

  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) mbar_init(&full[s], 1);
    mbar_fence_init();
    s_ndead = 0;
  }
  for (int t = tid; t < S; t += NT) {
    occl[t] = t;
    posv[t] = (t < n_loc) ? p.pos[(size_t)b * p.cap + s_begin + t] : 0;
  }
  for (int t = tid; t < CHUNK_TOKENS * H; t += NT) {
    const int i = t / H, h = t % H;
    const float2 e = (i < p.C) ? p.rt[((size_t)b * H + h) * CHUNK_TOKENS + i] : make_float2(0.f, 1.f);
    Rs[t] = e.x;
    Ts[t] = e.y;
  }
  __syncthreads();
  for (int h = tid; h < H; h += NT) {                        // token 0: nothing has been dropped yet
    hc[h] = -Rs[h] - __log2f(Ts[h] * (float)H);
    if (r == 0) p.ml[((size_t)b * H + h) * CHUNK_TOKENS] = make_float2(Rs[h], Ts[h]);
  }
  // logits of token i into buffer i % nstage: per head the CTA's state columns and the chunk's columns, 2 H bulk
  // copies shared out among the warps (a lane issues its copies one after the other: one warp alone would spend
  // more time issuing them than the token's arithmetic takes).  `arm` comes first, from one thread.
  auto arm = [&](int i) { mbar_expect_tx(&full[i % nstage], (uint32_t)H * (uint32_t)SW * 4u); };
  auto request = [&](int i) {
    uint64_t* bar = &full[i % nstage];
    float* dst = stage + (size_t)(i % nstage) * H * SW;
    const float* src = lgb + (size_t)i * H * p.ldc;
    if (lane < 4) {
      for (int j = warp * 4 + lane; j < 2 * H; j += NW * 4) {
        const int h = j >> 1;
        if (j & 1) bulk_g2s(dst + (size_t)h * SW + S, src + (size_t)h * p.ldc + p.capA, (uint32_t)CHUNK_TOKENS * 4u, bar);
        else bulk_g2s(dst + (size_t)h * SW, src + (size_t)h * p.ldc + s_begin, (uint32_t)S * 4u, bar);
      }
    }
  };
  if (tid == 0)
    for (int i = 0; i < min(nstage, p.C); ++i) arm(i);
  __syncthreads();
  for (int i = 0; i < min(nstage, p.C); ++i) request(i);
  cl.sync();                                                  // every CTA of the cluster runs: its shared memory may be written

  bool ok = true;
  for (int i = 0; i < p.C; ++i) {
    const int pos_i = first + i;
    const int par = i & 1;
    const bool more = i + 1 < p.C;
    const float* st = stage + (size_t)(i % nstage) * H * SW;
    const float* st1 = stage + (size_t)((i + 1) % nstage) * H * SW;   // the next token's logits (more)
    ok = warp_wait(&full[i % nstage], (uint32_t)((i / nstage) & 1)) && ok;
    // ---- head-averaged weight of this CTA's candidates, lowest (value, slot) -----------------------------
    float val = INFINITY;
    int idx = 0x7fffffff, ccol = -1;
    for (int t = tid; t < n_cand; t += NT) {
      const int c = (t < n_loc) ? occl[t] : S + i;
      const int pj = (t < n_loc) ? posv[t] : pos_i;
      const float* col = st + c;
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;       // fixed order: heads h = 0,4,8,.. / 1,5,.. / 2,6,.. / 3,7,..
      int h = 0;
      for (; h + 7 < H; h += 8) {                         // eight heads' logits requested before the first is used
        float x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = col[(h + u) * SW] + hc[h + u];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = exp2_fast(x[u]);
        a0 += x[0] + x[4];
        a1 += x[1] + x[5];
        a2 += x[2] + x[6];
        a3 += x[3] + x[7];
      }
      for (; h < H; ++h) a0 += exp2_fast(col[h * SW] + hc[h]);
      float a = (a0 + a1) + (a2 + a3);
      if (p.window) a = (float)(pj - pos_i);             // Window: the earliest position goes
      if (pj < p.keep_first) a = INFINITY;
      const int g = (t < n_loc) ? s_begin + t : p.cap;
      if (a < val) { val = a; idx = g; ccol = c; }      // t ascends and with it the slot: strict < keeps the lowest
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, val, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      const int oc = __shfl_xor_sync(0xffffffffu, ccol, o);
      if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; ccol = oc; }
    }
    if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; red_c[warp] = ccol; }
    // ---- this CTA's correction for token i+1: the terms of the columns that died in its care so far --------
    if (more) {
      ok = warp_wait(&full[(i + 1) % nstage], (uint32_t)(((i + 1) / nstage) & 1)) && ok;
      const int nd = s_ndead;
      for (int h = warp; h < H; h += NW) {                  // a warp per head, a lane per dead column
        const float R1 = Rs[(i + 1) * H + h];
        float g = 0.f;
        for (int d = lane; d < nd; d += 32) g += exp2_fast(st1[h * SW + dead[d]] - R1);
        g = warp_sum(g);
        if (lane == 0) s_co[h] = g;
      }
    }
    __syncthreads();
    if (warp == 0) {
      val = (lane < NW) ? red_v[lane] : INFINITY;
      idx = (lane < NW) ? red_i[lane] : 0x7fffffff;
      ccol = (lane < NW) ? red_c[lane] : -1;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, val, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        const int oc = __shfl_xor_sync(0xffffffffu, ccol, o);
        if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; ccol = oc; }
      }
      // the candidate to every CTA, and with it what the next token's normaliser loses if this candidate is the
      // one to go (its terms for token i+1) and this CTA's correction
      if (lane < NC) *cl.map_shared_rank(&best[par][r], lane) = make_float2(val, __int_as_float(idx));
      if (more) {
        for (int h = lane; h < H; h += 32) {
          const float en = (ccol >= 0) ? exp2_fast(st1[h * SW + ccol] - Rs[(i + 1) * H + h]) : 0.f;
          const float co = s_co[h];
          for (int q = 0; q < NC; ++q) {
            *cl.map_shared_rank(&xen[((size_t)par * NCM + r) * H + h], q) = en;
            *cl.map_shared_rank(&xco[((size_t)par * NCM + r) * H + h], q) = co;
          }
        }
      }
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    // ---- the same arg-min in every CTA; the slot's owner lets the token in; the next token's normaliser ----------
    float bv = INFINITY;
    int bi = 0x7fffffff, rw = 0;
    for (int rr = 0; rr < NC; ++rr) {
      const float2 e = best[par][rr];
      const int ei = __float_as_int(e.y);
      if (e.x < bv || (e.x == bv && ei < bi)) { bv = e.x; bi = ei; rw = rr; }
    }
    if (bi < 0 || bi > p.cap) {                          // cannot happen with finite logits: report, drop the token
      if (tid == 0 && r == 0) atomicExch(p.status, DEV_ERR_BAD_VICTIM);
      bi = p.cap;
      rw = 0;
    }
    if (more) {
      for (int h = tid; h < H; h += NT) {
        float gone = xen[((size_t)par * NCM + rw) * H + h];
        for (int rr = 0; rr < NC; ++rr) gone += xco[((size_t)par * NCM + rr) * H + h];
        const float R1 = Rs[(i + 1) * H + h];
        const float L = Ts[(i + 1) * H + h] - gone;
        hc[h] = -R1 - __log2f(L * (float)H);
        if (r == 0) p.ml[((size_t)b * H + h) * CHUNK_TOKENS + i + 1] = make_float2(R1, L);
      }
    }
    if (tid == 0) {
      if (i + nstage < p.C) arm(i + nstage);             // (this buffer's phase of token i was consumed above)
      if (bi < p.cap) {
        const int l = bi - s_begin;
        if (l >= 0 && l < n_loc) {                      // Eq. 9 in place: the token takes the dropped row's slot
          const int old = occl[l];
          p.death[(size_t)b * p.ldc + (old < S ? s_begin + old : p.capA + (old - S))] = i;
          if (p.evicted) p.evicted[(size_t)i * p.B + b] = posv[l];
          occl[l] = S + i;
          posv[l] = pos_i;
          dead[s_ndead] = old;
          s_ndead = s_ndead + 1;
        }
      } else if (r == 0) {                               // the token itself had the lowest weight
        p.death[(size_t)b * p.ldc + p.capA + i] = i;
        if (p.evicted) p.evicted[(size_t)i * p.B + b] = pos_i;
        dead[s_ndead] = S + i;
        s_ndead = s_ndead + 1;
      }
    }
    __syncthreads();                                     // the buffer has been read by everybody; occl, hc, dead are up to date
    if (i + nstage < p.C) {
      fence_proxy_async_smem();
      request(i + nstage);
    }
  }
  if (!ok && tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
  for (int t = tid; t < n_loc; t += NT) {
    p.pos[(size_t)b * p.cap + s_begin + t] = posv[t];
    p.slot_token[(size_t)b * p.cap + s_begin + t] = (occl[t] >= S) ? occl[t] - S : -1;
  }
}

// Rows of the chunk's surviving tokens into the slots they took; bookkeeping for the kernels that follow
// (a plain launch: a later streaming kernel, which requests rows before its own dependency wait, starts only
// once these copies are complete; no single "last written row" exists, so that hint is cleared).
template <int D>
__global__ void tova_chunk_scatter_kernel(const ChunkParams p) {
  constexpr int CH = D * 2 / 16;
  const size_t total = (size_t)p.B * p.cap * p.Hkv * CH;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int ch = (int)(i % CH);
    const size_t r = i / CH;                           // (b, s, kvh)
    const int kvh = (int)(r % p.Hkv);
    const size_t bs = r / p.Hkv;                       // b * cap + s
    const int t = p.slot_token[bs];
    if (t < 0) continue;
    const int b = (int)(bs / p.cap), s = (int)(bs % p.cap);
    const size_t src = (((size_t)b * p.Hkv + kvh) * CHUNK_TOKENS + t) * CH + ch;
    const size_t dst = (((size_t)b * p.Hkv + kvh) * p.cap + s) * CH + ch;
    reinterpret_cast<uint4*>(p.K)[dst] = reinterpret_cast<const uint4*>(p.Kst)[src];
    reinterpret_cast<uint4*>(p.V)[dst] = reinterpret_cast<const uint4*>(p.Vst)[src];
  }
  if (blockIdx.x == 0) {
    for (int b = threadIdx.x; b < p.B; b += blockDim.x) p.last_slot[b] = -1;
    if (threadIdx.x == 0) *p.cur_pos = *p.first + p.C - 1;
  }
}

}  // namespace tova
