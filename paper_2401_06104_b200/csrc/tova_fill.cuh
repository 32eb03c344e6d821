// Bulk fill of the multi-state (sm_100a): while the state has free rows, g(t) = min(t, k)
// (Section 3.3) is not reached and no token is dropped, so a run of F prompt tokens that
// all fit behaves like ordinary causal attention: token i of the run attends to the n0
// rows already held plus tokens 0..i of the run (Eq. 6 appends before Eq. 7 attends), and
// every token of the run stays.  Instead of F dependent decode steps, three launches:
//
//   tova_fill_rows_kernel    copies the run's keys/values into rows n0..n0+F-1 of the
//                            state and records their positions (evicted position = -1);
//   tova_fill_attn_kernel    causal attention of the run's queries over the state (dense
//                            contraction: warp-level bf16 tensor-core MMAs, fp32 softmax);
//   tova_fill_commit_kernel  length, last written row and current position.
//
// The attention kernel: one CTA of 4 warps per (64 query tokens, query head, sequence);
// a warp owns 16 query rows.  Key/value tiles of 64 rows arrive by tiled TMA
// (cp.async.bulk.tensor.2d, 128-byte swizzle) into a two-stage ring and are read with
// ldmatrix; S = Q K^T and O += P V as mma.sync.m16n8k16 bf16 -> fp32; the soft-max
// weights enter the second contraction as hi + lo (two bf16 terms), like the decode
// kernel's.  Logits are kept in the base-2 domain (scale2 = sm_scale * log2 e).
#pragma once

#include <cuda.h>

#include "tova_device.cuh"
#include "tova_split_mma.cuh"

namespace tova {

constexpr int FILL_Q_ROWS = 64;    // query tokens per CTA
constexpr int FILL_K_ROWS = 64;    // state rows per tile
constexpr int FILL_THREADS = 128;

struct FillParams {
  unsigned char* K;        // [B,Hkv,cap,D] state
  unsigned char* V;
  int32_t* pos;            // [B,cap]
  int32_t* len;            // [B]
  int32_t* last_slot;      // [B]
  int32_t* cur_pos;        // [1]
  int32_t* status;         // [1]
  const void* q;           // [F,B,H,D]
  const void* k_new;       // [F,B,Hkv,D]
  const void* v_new;
  float* out;              // [F,B,H,D]
  int32_t* evicted;        // [F,B] ([F,B,units] with per-unit tables) or null
  int32_t* upos;           // [B,units,cap] per-unit slot tables (head-wise TOVA), or null
  int units;               // units that own rows: 1 (the layer) or Hkv
  int B, H, Hkv, G, cap;
  int n0;                  // rows held before the run
  int F;                   // tokens in the run (n0 + F <= cap)
  int first_pos;           // position of the run's first token, or < 0: current position + 1
  float scale2;
};

// Rows of the run into the state, their positions, "nothing dropped".
// grid.x covers F*B*Hkv rows of 16-byte chunks; any 1-D launch works (grid-stride).
template <int D>
__global__ void tova_fill_rows_kernel(const FillParams p) {
  constexpr int CH = D * 2 / 16;   // 16-byte chunks per bf16 row
  const int first = (p.first_pos < 0) ? *p.cur_pos + 1 : p.first_pos;
  const size_t total = (size_t)p.F * p.B * p.Hkv * CH;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int ch = (int)(i % CH);
    const size_t row = i / CH;                 // (t, b, kvh) in input order
    const int kvh = (int)(row % p.Hkv);
    const int b = (int)((row / p.Hkv) % p.B);
    const int t = (int)(row / ((size_t)p.Hkv * p.B));
    const size_t dst = (((size_t)b * p.Hkv + kvh) * p.cap + p.n0 + t) * CH + ch;
    reinterpret_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[i];
    reinterpret_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[i];
  }
  const size_t tb = (size_t)p.F * p.B;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < tb; i += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(i % p.B);
    const int t = (int)(i / p.B);
    p.pos[(size_t)b * p.cap + p.n0 + t] = first + t;
    if (p.upos) {                      // every unit holds the same tokens while nothing is dropped
      for (int u = 0; u < p.units; ++u) {
        p.upos[((size_t)b * p.units + u) * p.cap + p.n0 + t] = first + t;
        if (p.evicted) p.evicted[i * p.units + u] = -1;
      }
    } else if (p.evicted) {
      p.evicted[i] = -1;
    }
  }
}

__global__ void tova_fill_commit_kernel(const FillParams p) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < p.B) {
    p.len[i] = p.n0 + p.F;
    p.last_slot[i] = p.n0 + p.F - 1;
  }
  if (i == 0) *p.cur_pos = ((p.first_pos < 0) ? *p.cur_pos + 1 : p.first_pos) + p.F - 1;
}

// Tiled TMA load without a cache hint: the tiles of a head are read again by the other query tiles
// and by the other heads of its group, so they should stay in L2.
__device__ __forceinline__ void tma_load_2d_keep(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_addr(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_addr(bar))
      : "memory");
}

// Byte offset of 16-byte chunk `chunk` (0..D/8-1) of row `row` (0..63) in a tile stored as
// D/64 boxes of [64 rows][128 bytes] with the 128-byte swizzle (boxes 1024-byte aligned).
__device__ __forceinline__ uint32_t fill_swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * (FILL_K_ROWS * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// grid = (ceil(F/64), H, B), block = 128.  Dynamic shared memory: 2 x (K tile + V tile) + 1 KiB slack; three CTAs per SM.
template <int D>
__global__ void __launch_bounds__(FILL_THREADS, 3) tova_fill_attn_kernel(const FillParams p,
                                                                      const __grid_constant__ CUtensorMap map_k,
                                                                      const __grid_constant__ CUtensorMap map_v) {
  constexpr int TILE_BYTES = FILL_K_ROWS * D * 2;  // 8 KiB (D=64) or 16 KiB (D=128)
  constexpr int BOXES = D / 64;
  constexpr int KS = D / 16;                       // k-steps of Q K^T
  constexpr int ND = D / 8;                        // n-tiles of P V

  extern __shared__ unsigned char fill_smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(fill_smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* kv_s = smem;                              // stage s: K at 2s, V at 2s+1
  __shared__ __align__(8) uint64_t bars[2];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile_q = gridDim.x - 1 - blockIdx.x;           // longest rows first
  const int t0 = tile_q * FILL_Q_ROWS;
  const int h = blockIdx.y, b = blockIdx.z;
  const int kvh = h / p.G;
  const int head_row0 = (b * p.Hkv + kvh) * p.cap;         // first row of this head in the [B*Hkv*cap, D] view
  const int t_last = min(t0 + FILL_Q_ROWS, p.F) - 1;       // last real token of this CTA
  const int n_keys = p.n0 + t_last + 1;                    // rows visible to it
  const int n_tiles = (n_keys + FILL_K_ROWS - 1) / FILL_K_ROWS;

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
    mbar_expect_tx(bar, 2u * TILE_BYTES);
    const int y = head_row0 + i * FILL_K_ROWS;
#pragma unroll
    for (int bx = 0; bx < BOXES; ++bx) {
      tma_load_2d_keep(kd + bx * (FILL_K_ROWS * 128), &map_k, bx * 64, y, bar);
      tma_load_2d_keep(vd + bx * (FILL_K_ROWS * 128), &map_v, bx * 64, y, bar);
    }
  };
  if (tid == 0) issue(0);

  // A fragments of this warp's 16 query rows straight from global memory (every 32-byte sector is used in
  // full), kept in registers for the whole kernel; rows past the run repeat its last token.
  uint32_t qa[KS][4];
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q);
    const int ra = min(t0 + warp * 16 + (lane >> 2), p.F - 1), rb = min(t0 + warp * 16 + (lane >> 2) + 8, p.F - 1);
    const uint32_t* qra = reinterpret_cast<const uint32_t*>(qg + (((size_t)ra * p.B + b) * p.H + h) * D) + (lane & 3);
    const uint32_t* qrb = reinterpret_cast<const uint32_t*>(qg + (((size_t)rb * p.B + b) * p.H + h) * D) + (lane & 3);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = __ldg(qra + ks * 8);
      qa[ks][1] = __ldg(qrb + ks * 8);
      qa[ks][2] = __ldg(qra + ks * 8 + 4);
      qa[ks][3] = __ldg(qrb + ks * 8 + 4);
    }
  }

  float o[ND][4];
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};   // rows lane/4 and lane/4 + 8
  float l_run[2] = {0.f, 0.f};               // this lane's share of the row sums

  const int row_lo = warp * 16 + (lane >> 2);
  // last visible state row of this lane's two query rows (rows past the run see what its last token sees)
  const int vis0 = p.n0 + min(t0 + row_lo, p.F - 1);
  const int vis1 = p.n0 + min(t0 + row_lo + 8, p.F - 1);
  bool ok = true;

  for (int i = 0; i < n_tiles; ++i) {
    if (tid == 0 && i + 1 < n_tiles) issue(i + 1);   // its buffers were released by the barrier ending tile i-1
    ok = warp_wait(&bars[i & 1], (uint32_t)((i >> 1) & 1)) && ok;
    const uint32_t kt = smem_addr(kv_s + (size_t)(2 * (i & 1)) * TILE_BYTES);
    const uint32_t vt = kt + TILE_BYTES;
    const int j0 = i * FILL_K_ROWS;

    // S[16 x 64] = Q K^T
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

    // scale, causal mask, running max
    const bool need_mask = j0 + FILL_K_ROWS - 1 > p.n0 + t0;   // some row of the CTA cannot see the whole tile
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int j = j0 + nt * 8 + 2 * (lane & 3);
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float a = s[nt][e] * p.scale2, c = s[nt][2 + e] * p.scale2;
        if (need_mask) {
          if (j + e > vis0) a = -INFINITY;
          if (j + e > vis1) c = -INFINITY;
        }
        s[nt][e] = a;
        s[nt][2 + e] = c;
        mx0 = fmaxf(mx0, a);
        mx1 = fmaxf(mx1, c);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
    // A row that sees nothing of this tile keeps its state (mn stays -inf only before its first visible tile,
    // and tile 0 always holds row 0, visible to every query).
    const float c0 = exp2_diff(m_run[0], mn0), c1 = exp2_diff(m_run[1], mn1);
    m_run[0] = mn0;
    m_run[1] = mn1;
    l_run[0] *= c0;
    l_run[1] *= c1;
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) {
      o[nd][0] *= c0; o[nd][1] *= c0;
      o[nd][2] *= c1; o[nd][3] *= c1;
    }
    const float b0 = (mn0 == -INFINITY) ? 0.f : mn0, b1 = (mn1 == -INFINITY) ? 0.f : mn1;

    // P = exp2(S - m), as A fragments (hi + lo); O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t ph[4], pl[4];
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int nt = 2 * kk + half;
        const float e0 = exp2f(s[nt][0] - b0), e1 = exp2f(s[nt][1] - b0);
        const float e2 = exp2f(s[nt][2] - b1), e3 = exp2f(s[nt][3] - b1);
        l_run[0] += e0 + e1;
        l_run[1] += e2 + e3;
        split_hi_lo(e0, e1, ph[2 * half], pl[2 * half]);
        split_hi_lo(e2, e3, ph[2 * half + 1], pl[2 * half + 1]);
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
    fence_proxy_async_smem();   // this tile's reads are ordered before the copy that reuses its buffers
    __syncthreads();
  }

  if (!ok) {
    if (tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    return;
  }

  // row sums across the quad, normalise, store
  float l0 = l_run[0], l1 = l_run[1];
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float r0 = 1.f / l0, r1 = 1.f / l1;
  const int ta = t0 + row_lo, tb = ta + 8;
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) {
    const int d = nd * 8 + 2 * (lane & 3);
    if (ta < p.F)
      *reinterpret_cast<float2*>(p.out + (((size_t)ta * p.B + b) * p.H + h) * D + d) =
          make_float2(o[nd][0] * r0, o[nd][1] * r0);
    if (tb < p.F)
      *reinterpret_cast<float2*>(p.out + (((size_t)tb * p.B + b) * p.H + h) * D + d) =
          make_float2(o[nd][2] * r1, o[nd][3] * r1);
  }
}

}  // namespace tova
