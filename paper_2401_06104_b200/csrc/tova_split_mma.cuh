// Split kernel for grouped-query attention on tensor cores (bf16 state).
//
// With G >= 4 query heads sharing a KV head, the logits of a tile are a real
// dense contraction and so is the weighted sum (Eq. 4, Eq. 7).  One warp per
// (sequence, KV head, chunk) runs them as m16n8k16 bf16 MMAs with fp32
// accumulation, in the transposed form that keeps the MMA tile full:
//   S^T[rows, heads] = K[rows, D] . q^T[D, heads]      M = the tile's 16 rows, N = 8 heads
//   O^T[D, heads]   += V^T[D, rows] . P^T[rows, heads] M = 16 of the D columns, N = 8 heads
// (a second N tile when the group has more than 8 heads).  K and V^T are the A
// operands, read from shared memory with ldmatrix (V transposed on the way);
// q^T stays in registers; P^T goes from the accumulator layout of S^T to the
// B-operand layout with four 8x8 warp transposes (movmatrix) per tile.
//   - K/V tiles of 16 rows arrive through tiled TMA copies (tensor maps with the
//     128-byte swizzle), so that ldmatrix reads them without bank conflicts;
//   - products of bf16 inputs are exact in fp32, so the logits match an fp32
//     evaluation up to summation order;
//   - the soft-max weights are split into two bf16 terms (p = hi + lo, 16
//     significant bits) before they multiply V, which keeps the output within
//     the tolerance an fp32 weight would give.
// Same scratch outputs as the generic split kernel: logits, one (max, sum,
// weighted V sum) partial per head and chunk.
#pragma once

#include <cuda.h>

#include "tova_kernels.cuh"

namespace tova {

constexpr int MMA_UNIT_HEADS = 16;  // query heads one MMA split warp carries

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
      "%3}], [%4], %5;" ::"r"(smem_addr(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_addr(bar)), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// D += A (16x16, row) * B (16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Transposes an 8x8 matrix of 16-bit elements held one row pair per lane (lane = 4*row + col/2):
// afterwards the lane holds elements (2(lane%4), lane/4) and (2(lane%4)+1, lane/4) of the input.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// (x, y) -> bf16x2 with x in the low half; and the rounding remainders.
__device__ __forceinline__ void split_hi_lo(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - __low2float(h), y - __high2float(h));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Byte offset of the 16-byte chunk `chunk` (0..D/8-1) of row `row` (0..15) in
// a tile stored as D/64 boxes of [16 rows][128 bytes] with the 128-byte swizzle.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * (TILE_ROWS * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// grid = (max(n_chunks,1), Hkv*hgroups, B), block = one warp.
// TWO: the group has more than 8 heads, rows 8..15 of the MMA tile are in use.
template <int D, bool TWO, bool FUSED>
__global__ void __launch_bounds__(FUSED ? 32 * SPLIT_MERGE_MAX_WARPS : 32, FUSED ? (TWO ? 1 : 2) : 0) tova_split_mma_kernel(const StepParams p,
                                                            const __grid_constant__ CUtensorMap map_k,
                                                            const __grid_constant__ CUtensorMap map_v) {
  using T = __nv_bfloat16;
  constexpr int RB = D * 2;
  constexpr int TILE_BYTES = TILE_ROWS * RB;   // 2 KiB (D=64) or 4 KiB (D=128): a multiple of the swizzle period
  constexpr int NBOX = D / 64;
  constexpr int NB = SPLIT_BUFFERS;
  constexpr int KS = D / 16;                   // k-steps of q.K^T, and pairs of n-tiles of P.V
  constexpr int EPL = 8, LPR = RB / 16;

  extern __shared__ unsigned char smem_raw[];
  // the swizzle is a function of the shared-memory address: tiles start on 1 KiB boundaries
  constexpr int WARP_SMEM = NB * TILE_BYTES;   // per warp; a multiple of 1 KiB
  const int wib = FUSED ? threadIdx.y : 0;     // warp in block (FUSED: one CTA per head group, one warp per chunk)
  unsigned char* ring0 = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  unsigned char* ring = ring0 + (size_t)wib * WARP_SMEM;
  __shared__ __align__(8) uint64_t bars_all[SPLIT_MERGE_MAX_WARPS][NB];
  uint64_t* bars = bars_all[wib];
  const float* part0 = reinterpret_cast<const float*>(ring0);      // warp 0's partial
  __shared__ float snew_s[MMA_UNIT_HEADS];                         // the new token's logit per head (chunk 0's warp)
  // merge_ctas > 1: this CTA's inbox for the cluster merge, behind the rings
  float* cpart = reinterpret_cast<float*>(ring0 + (size_t)(FUSED ? blockDim.y : 1) * WARP_SMEM);
  // fuse_out: once all tiles are consumed the ring holds this warp's partial
  // [MMA_UNIT_HEADS][D+4] and (rank 0) the new token's logits
  float* part = reinterpret_cast<float*>(ring);
  static_assert((MMA_UNIT_HEADS * (D + PART_STRIDE_EXTRA) + MMA_UNIT_HEADS) * sizeof(float) <= (size_t)NB * TILE_BYTES,
                "partial fits the ring");

  // Merge across a cluster: peers will store into this CTA's shared memory; report in (see cluster_merge_outputs).
  if (FUSED && p.merge_ctas > 1) cluster_arrive_release();

  const int lane = threadIdx.x;
  const int qrow = lane >> 2, qcol = (lane & 3) * 2;   // fragment coordinates of this lane
  const int c = FUSED ? (int)(blockIdx.x * blockDim.y) + wib : (int)blockIdx.x, b = blockIdx.z;
  const int kvh = blockIdx.y / p.hgroups, hg = blockIdx.y % p.hgroups;
  const int g_begin = hg * MMA_UNIT_HEADS;
  const int g_cnt = min(MMA_UNIT_HEADS, p.G - g_begin);
  constexpr int R = TWO ? 2 : 1;                        // 8-row halves of the MMA tile that hold heads
  const int row_begin = c * p.chunk_rows;
  const int rows = min(max(p.n - row_begin, 0), p.chunk_rows);
  const int ntiles = (rows + TILE_ROWS - 1) / TILE_ROWS;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < NB; ++s) mbar_init(&bars[s], 1);
    mbar_fence_init();
  }
  __syncwarp();

  const int y0 = ((b * p.Hkv + kvh) * p.cap) + row_begin;   // first row of the chunk in the [rows, D] view
  const int n_ops = 2 * ntiles;                             // u = 2t: K_t, u = 2t+1: V_t
  const uint64_t stream_policy = l2_policy_evict_first();   // K/V rows are read once per step
  auto issue = [&](int u) {                                 // lane 0 only
    uint64_t* bar = &bars[u % NB];
    unsigned char* dst = ring + (size_t)(u % NB) * TILE_BYTES;
    mbar_expect_tx(bar, TILE_BYTES);                        // a tiled copy always delivers the whole box
#pragma unroll
    for (int bx = 0; bx < NBOX; ++bx)
      tma_load_2d(dst + bx * (TILE_ROWS * 128), (u & 1) ? &map_v : &map_k, bx * 64, y0 + (u >> 1) * TILE_ROWS, bar,
                  stream_policy);
  };
  // Early prefetch before the dependency wait: only the row the previous step's
  // token went to (last_slot) can still change; it is fetched again after the
  // wait if it lies in the tiles requested here.
  const bool early = p.last_slot != nullptr;
  if (early && lane == 0) {
    for (int u = 0; u < min(NB, n_ops); ++u) issue(u);
  }

  pdl_wait();
  pdl_launch_dependents();

  if (c == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0)
    *p.cur_pos = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;
  if (!early && lane == 0) {
    for (int u = 0; u < min(NB, n_ops); ++u) issue(u);
  }
  // Every global load of the prologue is issued before the first one is used:
  // the row that may have changed, q^T (the B operand of S^T = K . q^T) and, for
  // chunk 0's warp, the new token's key and the q rows in the layout of its dot products.
  const T* qbase = static_cast<const T*>(p.q) + ((size_t)b * p.H + (size_t)kvh * p.G + g_begin) * D;
  const size_t bh0 = (size_t)b * p.H + (size_t)kvh * p.G + g_begin;
  const int ls = early ? __ldcg(p.last_slot + b) : -1;
  // q^T: column n of the MMA tile is head n (heads beyond the group are zero), 16 of the D values per k-step.
  // qb[ks][2*nh + {0,1}]: head-tile nh (heads 8nh..8nh+7), d = 16ks + qcol (+8)
  uint32_t qb[KS][2 * R];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const int d = ks * 16 + qcol;
#pragma unroll
    for (int nh = 0; nh < R; ++nh) {
      const int head = qrow + 8 * nh;
      const uint32_t* r = reinterpret_cast<const uint32_t*>(qbase + (size_t)head * D + d);
      qb[ks][2 * nh] = (head < g_cnt) ? r[0] : 0u;
      qb[ks][2 * nh + 1] = (head < g_cnt) ? r[4] : 0u;   // d + 8
    }
  }
  constexpr int HPP = 32 / LPR;                       // heads per pass of the new token's dot products
  constexpr int NPASS = (TWO ? 16 : 8) / HPP;
  const int lig = lane % LPR, hsub = lane / LPR;
  uint4 knw = make_uint4(0u, 0u, 0u, 0u), qw[NPASS];
  if (c == 0) {
    knw = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.k_new) + ((size_t)b * p.Hkv + kvh) * D + lig * EPL);
#pragma unroll
    for (int ps = 0; ps < NPASS; ++ps) {
      const int g = ps * HPP + hsub;
      qw[ps] = *reinterpret_cast<const uint4*>(qbase + (size_t)min(g, g_cnt - 1) * D + lig * EPL);
    }
  }

  int patch_row = -1;
  if (ls >= row_begin && ls < row_begin + rows) patch_row = ls - row_begin;
  const unsigned char* k_rows = static_cast<const unsigned char*>(p.K) + (size_t)y0 * RB;
  const unsigned char* v_rows = static_cast<const unsigned char*>(p.V) + (size_t)y0 * RB;
  // Re-fetches row patch_row of operand tile u (already landed) into the swizzled tile.
  auto patch = [&](int u, const unsigned char* src) {
    if (patch_row >= 0 && u < NB && patch_row / TILE_ROWS == (u >> 1)) {
      if (lane < LPR) {
        const uint4 w = __ldcg(reinterpret_cast<const uint4*>(src + (size_t)patch_row * RB) + lane);
        *reinterpret_cast<uint4*>(ring + (size_t)(u % NB) * TILE_BYTES + swz(patch_row % TILE_ROWS, lane)) = w;
      }
      __syncwarp();
    }
  };

  // The new token (candidate n): its logit per head, on the plain ALUs, HPP heads per pass.
  if (c == 0) {
    float kf[EPL];
    Vec16<T>::unpack(knw, kf);
#pragma unroll
    for (int ps = 0; ps < NPASS; ++ps) {
      if (ps * HPP < g_cnt) {
        const int g = ps * HPP + hsub;
        float qf[EPL];
        Vec16<T>::unpack(qw[ps], qf);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
        for (int o = LPR / 2; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= p.scale2;
        if (lig == 0 && g < g_cnt) {
          p.logits[(bh0 + g) * p.ld + p.n] = s;
          if (FUSED) snew_s[g] = s;
          else p.part_ml[(bh0 + g) * p.pc + p.n_chunks] = make_float2(s, 1.f);
        }
      }
    }
    if (FUSED && p.k_stage && hg == 0 && lane < LPR) {  // copies for a deferred eviction
      const size_t w16 = ((size_t)b * p.Hkv + kvh) * LPR + lane;
      static_cast<uint4*>(p.k_stage)[w16] = static_cast<const uint4*>(p.k_new)[w16];
      static_cast<uint4*>(p.v_stage)[w16] = static_cast<const uint4*>(p.v_new)[w16];
    }
  }
  if (ntiles == 0) {
    if (FUSED) {
      empty_partial<D>(part, MMA_UNIT_HEADS, lane);
      fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
    }
    return;
  }

  // O^T[D, heads]: accumulator tile (nh, mt) covers d = 16mt..16mt+15 of heads 8nh..8nh+7;
  // this lane holds d = 16mt + qrow (+8) of heads 8nh + qcol, qcol + 1
  float o[R][KS][4];
#pragma unroll
  for (int nh = 0; nh < R; ++nh)
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[nh][mt][e] = 0.f;
  float m[R][2], l[R][2];   // heads 8nh + qcol + {0,1}
#pragma unroll
  for (int nh = 0; nh < R; ++nh) {
    m[nh][0] = m[nh][1] = -INFINITY;
    l[nh][0] = l[nh][1] = 0.f;
  }

  // ldmatrix lane roles: lane supplies the address of row (lane % 8) of matrix (lane / 8)
  const int lm_r = lane & 7, lm_m = lane >> 3;
  const uint32_t ring_addr = smem_addr(ring);
  // swz(row, 2i + c) with this lane's row and c, for the four values of i mod 4, worked out once:
  // the 16-byte column 2(i mod 4) + c is XORed with row mod 8 = lm_r, and 2(i mod 4) has no bit in
  // common with c, so the lane-dependent part (c ^ lm_r) << 4 splits off.
  uint32_t k_ofs[4], v_ofs[4];   // K: row lm_r + 8(lm_m & 1), c = lm_m >> 1;  V: row lm_r + 8(lm_m >> 1), c = lm_m & 1
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    k_ofs[a] = (uint32_t)(lm_r + 8 * (lm_m & 1)) * 128u + ((uint32_t)(a * 32) ^ ((uint32_t)(((lm_m >> 1) ^ lm_r) & 7) << 4));
    v_ofs[a] = (uint32_t)(lm_r + 8 * (lm_m >> 1)) * 128u + ((uint32_t)(a * 32) ^ ((uint32_t)(((lm_m & 1) ^ lm_r) & 7) << 4));
  }

  bool failed = false;
  int t = 0;
  for (; t < ntiles; ++t) {
    const int uk = 2 * t, uv = 2 * t + 1;
    const int nvalid = min(TILE_ROWS, rows - t * TILE_ROWS);
    const uint32_t kt = ring_addr + (uint32_t)(uk % NB) * TILE_BYTES;
    const uint32_t vt = ring_addr + (uint32_t)(uv % NB) * TILE_BYTES;

    // ---- S^T = K . q^T: the tile's 16 rows are the M rows of the MMA -------------
    if (!warp_wait(&bars[uk % NB], (uint32_t)(uk / NB) & 1u)) { failed = true; break; }
    patch(uk, k_rows);
    float s[R][4];    // rows qrow (e = 0,1) and qrow + 8 (e = 2,3) of heads 8nh + qcol + (e & 1)
#pragma unroll
    for (int nh = 0; nh < R; ++nh)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[nh][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      // A fragment: (rows 0-7, d0..7) (rows 8-15, d0..7) (rows 0-7, d0+8..15) (rows 8-15, d0+8..15)
      uint32_t ka[4];
      ldmatrix_x4(ka, kt + k_ofs[ks & 3] + (uint32_t)(ks >> 2) * (TILE_ROWS * 128));
#pragma unroll
      for (int nh = 0; nh < R; ++nh) mma_bf16(s[nh], ka, qb[ks][2 * nh], qb[ks][2 * nh + 1]);
    }
    __syncwarp();
    if (lane == 0 && uk + NB < n_ops) {
      fence_proxy_async_smem();
      issue(uk + NB);
    }

    // ---- online soft-max on the fragments ----------------------------------------
    const bool row_lo = qrow < nvalid, row_hi = qrow + 8 < nvalid;
    uint32_t pb_hi[R][2], pb_lo[R][2];   // P^T as the B operand of O^T += V^T . P^T: rows 2(lane%4)+{0,1} (+8), head lane/4
#pragma unroll
    for (int nh = 0; nh < R; ++nh) {
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = ((e < 2) ? row_lo : row_hi) ? s[nh][e] * p.scale2 : -INFINITY;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int head = 8 * nh + qcol + hh;
        if (head < g_cnt) {
          float* lg = p.logits + (bh0 + head) * p.ld + row_begin + t * TILE_ROWS + qrow;
          if (row_lo) lg[0] = v[hh];
          if (row_hi) lg[8] = v[2 + hh];
        }
      }
      float e4[4];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float mx = fmaxf(v[hh], v[2 + hh]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float m_new = fmaxf(m[nh][hh], mx);
        const float corr = exp2_diff(m[nh][hh], m_new);
        e4[hh] = exp2_diff(v[hh], m_new);
        e4[2 + hh] = exp2_diff(v[2 + hh], m_new);
        l[nh][hh] = fmaf(l[nh][hh], corr, e4[hh] + e4[2 + hh]);   // per-lane partial, folded at the end
        m[nh][hh] = m_new;
        if (__any_sync(0xffffffffu, corr != 1.f)) {   // the running max moved for some head: rescale (rare after the first tiles)
#pragma unroll
          for (int mt = 0; mt < KS; ++mt) {
            o[nh][mt][hh] *= corr;
            o[nh][mt][2 + hh] *= corr;
          }
        }
      }
      // weights as two bf16 terms, then from the accumulator layout (row = lane/4, heads
      // 2(lane%4)+{0,1}) to the B-operand layout (rows 2(lane%4)+{0,1}, head = lane/4)
      uint32_t hi0, lo0, hi1, lo1;
      split_hi_lo(e4[0], e4[1], hi0, lo0);   // rows 0-7
      split_hi_lo(e4[2], e4[3], hi1, lo1);   // rows 8-15
      pb_hi[nh][0] = movmatrix_trans(hi0);
      pb_hi[nh][1] = movmatrix_trans(hi1);
      pb_lo[nh][0] = movmatrix_trans(lo0);
      pb_lo[nh][1] = movmatrix_trans(lo1);
    }

    // ---- O^T += V^T . P^T ----------------------------------------------------------------
    if (!warp_wait(&bars[uv % NB], (uint32_t)(uv / NB) & 1u)) { failed = true; break; }
    patch(uv, v_rows);
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
      // A fragment of V^T (d rows, tile-row columns), transposing loads:
      // (rows 0-7, d0..7) (rows 0-7, d0+8..15) (rows 8-15, d0..7) (rows 8-15, d0+8..15)
      uint32_t va[4];
      ldmatrix_x4_trans(va, vt + v_ofs[mt & 3] + (uint32_t)(mt >> 2) * (TILE_ROWS * 128));
#pragma unroll
      for (int nh = 0; nh < R; ++nh) {
        mma_bf16(o[nh][mt], va, pb_hi[nh][0], pb_hi[nh][1]);
        mma_bf16(o[nh][mt], va, pb_lo[nh][0], pb_lo[nh][1]);
      }
    }
    __syncwarp();
    if (lane == 0 && uv + NB < n_ops) {
      fence_proxy_async_smem();
      issue(uv + NB);
    }
  }

  if (failed) {
    for (int u = 2 * t; u < min(2 * t + NB, n_ops); ++u) warp_wait(&bars[u % NB], (uint32_t)(u / NB) & 1u);
    if (lane == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    if (FUSED) {           // the other warps wait at the CTA barrier: join them with an empty partial
      empty_partial<D>(part, MMA_UNIT_HEADS, lane);
      fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
    }
    return;
  }

  // ---- chunk partial: (max, sum) and the un-normalised weighted V sums ------------------
  __syncwarp();                 // fuse_out: the partial goes where the tiles were
#pragma unroll
  for (int nh = 0; nh < R; ++nh)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int head = 8 * nh + qcol + hh;
      float lsum = l[nh][hh];
      lsum += __shfl_xor_sync(0xffffffffu, lsum, 4);
      lsum += __shfl_xor_sync(0xffffffffu, lsum, 8);
      lsum += __shfl_xor_sync(0xffffffffu, lsum, 16);
      if (head < g_cnt) {
        float* dst = FUSED ? part + head * (D + PART_STRIDE_EXTRA) + qrow
                           : p.part_acc + ((bh0 + head) * (size_t)(p.pc - 1) + c) * D + qrow;
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
          dst[mt * 16] = o[nh][mt][hh];
          dst[mt * 16 + 8] = o[nh][mt][2 + hh];
        }
        if (qrow == 0) {
          if (FUSED) {
            part[head * (D + PART_STRIDE_EXTRA) + D] = m[nh][hh];
            part[head * (D + PART_STRIDE_EXTRA) + D + 1] = lsum;
          } else {
            p.part_ml[(bh0 + head) * p.pc + c] = make_float2(m[nh][hh], lsum);
          }
        }
      }
    }
  if (FUSED) fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
}

}  // namespace tova
