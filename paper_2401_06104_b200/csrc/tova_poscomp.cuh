// Position compression for streams longer than the training context (sm_100a;
// Section "Extrapolation with TOVA").  Keys are cached WITHOUT rotary
// embedding.  At every step the retained tokens and the new token, in position
// order, get new positions in which a gap g between neighbours becomes
// ln(ln(g)), or stays g while g <= 10; the rotary embedding (rotate-half pairs
// d, d + D/2; angle p' * base^(-2d/D)) is applied with those positions to the
// cached keys as they are streamed and to the query; everything after the
// logits - soft-max, output, head average, arg-min, in-place insert - is the
// ordinary step.  Attention depends on differences of positions only, so the
// earliest retained token is put at 0.
//
//   tova_poscomp_kernel     per sequence: rank of every candidate by position,
//                           the chain of compressed positions (in double, summed
//                           in position order), a (cos, sin) table per candidate
//                           and frequency, and the rotated query in fp32;
//   tova_split_rope_kernel  the streaming kernel of this mode: one warp per
//                           (sequence, KV head, group of up to 4 query heads,
//                           chunk of rows); rows come by plain 16-byte loads,
//                           are rotated with the table (the partner component
//                           of a pair sits in another lane: one shuffle), then
//                           logits, online soft-max and weighted V sum on the
//                           plain ALUs; partials and logits go to the same
//                           scratch as the other streaming kernels', and the
//                           combine kernel finishes the step.
// This mode trades speed for range: a table read and a rotation per cached row
// and query-head group.  It is off unless the caller provides its workspace.
#pragma once

#include "tova_kernels.cuh"

namespace tova {

constexpr int POSCOMP_THREADS = 512;
constexpr int ROPE_UNIT_HEADS = 4;     // query heads one warp of the rotating streaming kernel carries

struct PosCompParams {
  float2* table;      // [B,cap+1,D/2] (cos, sin) of candidate j (slot order, the new token at index n) and frequency d
  float* q_rot;       // [B,H,D] the query after rotary embedding at the new token's compressed position
  double* cpos;       // [B,cap+1] compressed positions (kept for inspection)
  double rope_base;
};

__device__ __forceinline__ double compress_gap(int g) { return (g <= 10) ? (double)g : log(log((double)g)); }

// grid = (B), block = POSCOMP_THREADS.  Dynamic shared memory (poscomp_smem_bytes): per candidate a double (the
// chain) and three ints (position, rank, position by rank), plus D/2 doubles (inverse frequencies).
__host__ __device__ inline size_t poscomp_smem_bytes(int cap, int D) {
  return sizeof(double) * ((size_t)cap + 1 + D / 2) + sizeof(int32_t) * 3 * ((size_t)cap + 1);
}
template <typename T, int D>
__global__ void __launch_bounds__(POSCOMP_THREADS) tova_poscomp_kernel(const StepParams p, const PosCompParams pc) {
  constexpr int NT = POSCOMP_THREADS, HALF = D / 2;
  extern __shared__ __align__(16) unsigned char pcs_raw[];
  const int b = blockIdx.x, tid = threadIdx.x;
  const int m = p.n + 1;                                   // candidates: the live rows, then the new token
  double* chain = reinterpret_cast<double*>(pcs_raw);      // [m] compressed position by rank
  double* inv_freq = chain + m;                            // [HALF]
  int32_t* spos = reinterpret_cast<int32_t*>(inv_freq + HALF);   // [m] position by candidate
  int32_t* rank = spos + m;                                // [m] rank of the candidate in position order
  int32_t* sorted = rank + m;                              // [m] position by rank
  const int pos_t = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;    // the streaming kernel of this step updates cur_pos later

  for (int j = tid; j < m; j += NT) spos[j] = (j < p.n) ? p.pos[(size_t)b * p.cap + j] : pos_t;
  for (int d = tid; d < HALF; d += NT) inv_freq[d] = pow(pc.rope_base, -2.0 * (double)d / (double)D);
  __syncthreads();
  for (int j = tid; j < m; j += NT) {                      // positions are distinct: the rank is a permutation
    const int pj = spos[j];
    int r = 0;
    for (int i = 0; i < m; ++i) r += (spos[i] < pj || (spos[i] == pj && i < j)) ? 1 : 0;
    rank[j] = r;
  }
  __syncthreads();
  // positions by rank, then the compressed gap to the predecessor in position order
  for (int j = tid; j < m; j += NT) sorted[rank[j]] = spos[j];
  __syncthreads();
  for (int r = tid; r < m; r += NT) chain[r] = (r > 0) ? compress_gap(sorted[r] - sorted[r - 1]) : 0.0;
  __syncthreads();
  if (tid == 0) {                                          // the chain, summed in position order
    double acc = 0.0;
    for (int r = 0; r < m; ++r) {
      acc += chain[r];
      chain[r] = acc;
    }
  }
  __syncthreads();
  // table of (cos, sin) and the compressed positions, by candidate
  for (int j = tid; j < m; j += NT) pc.cpos[(size_t)b * (p.cap + 1) + j] = chain[rank[j]];
  float2* tab = pc.table + (size_t)b * (p.cap + 1) * HALF;
  for (int i = tid; i < m * HALF; i += NT) {
    const int j = i / HALF, d = i % HALF;
    double s, c;
    sincos(chain[rank[j]] * inv_freq[d], &s, &c);
    tab[i] = make_float2((float)c, (float)s);
  }
  __syncthreads();                                         // the new token's table row is complete (same block wrote it)
  // the query, rotated at the new token's position (fp32)
  const double pq = chain[rank[p.n]];
  for (int i = tid; i < p.H * HALF; i += NT) {
    const int h = i / HALF, d = i % HALF;
    double s, c;
    sincos(pq * inv_freq[d], &s, &c);
    const float cf = (float)c, sf = (float)s;
    const T* qh = static_cast<const T*>(p.q) + ((size_t)b * p.H + h) * D;
    const float a = (float)qh[d], bb = (float)qh[d + HALF];
    float* dst = pc.q_rot + ((size_t)b * p.H + h) * D;
    dst[d] = a * cf - bb * sf;
    dst[d + HALF] = bb * cf + a * sf;
  }
}

// grid = (max(n_chunks,1), Hkv*hgroups, B), block = one warp.  hgroups = ceil(G / ROPE_UNIT_HEADS).
template <typename T, int D>
__global__ void __launch_bounds__(32) tova_split_rope_kernel(const StepParams p, const PosCompParams pc) {
  constexpr int GU = ROPE_UNIT_HEADS;
  constexpr int EPL = Vec16<T>::N;          // elements per lane
  constexpr int RB = D * (int)sizeof(T);
  constexpr int LPR = RB / 16;              // lanes per row
  constexpr int RPW = 32 / LPR;             // rows per pass
  constexpr int HALF = D / 2;
  const int lane = threadIdx.x;
  const int lig = lane % LPR, sub = lane / LPR;
  const int c = blockIdx.x, b = blockIdx.z;
  const int kvh = blockIdx.y / p.hgroups, hg = blockIdx.y % p.hgroups;
  const int g_begin = hg * GU, g_cnt = min(GU, p.G - g_begin);
  const int row_begin = c * p.chunk_rows;
  const int rows = min(max(p.n - row_begin, 0), p.chunk_rows);
  const size_t bh0 = (size_t)b * p.H + (size_t)kvh * p.G + g_begin;
  const bool upper = lig >= LPR / 2;        // this lane holds components d + D/2 of the rotary pairs
  const int d0 = (lig % (LPR / 2)) * EPL;   // first frequency this lane needs

  if (c == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0)
    *p.cur_pos = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;

  // the rotated query of the unit's heads: this lane's EPL components per head
  float qf[GU][EPL];
#pragma unroll
  for (int g = 0; g < GU; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e) qf[g][e] = pc.q_rot[(bh0 + min(g, g_cnt - 1)) * D + lig * EPL + e];

  const float2* tab = pc.table + (size_t)b * (p.cap + 1) * HALF;
  // Rotates this lane's EPL components of a key row held by candidate j (raw 16 bytes in w).
  auto rotate = [&](const uint4& w, int j, float (&kf)[EPL]) {
    float own[EPL], oth[EPL];
    Vec16<T>::unpack(w, own);
    uint4 wo;
    wo.x = __shfl_xor_sync(0xffffffffu, w.x, LPR / 2);
    wo.y = __shfl_xor_sync(0xffffffffu, w.y, LPR / 2);
    wo.z = __shfl_xor_sync(0xffffffffu, w.z, LPR / 2);
    wo.w = __shfl_xor_sync(0xffffffffu, w.w, LPR / 2);
    Vec16<T>::unpack(wo, oth);
    const float2* tr = tab + (size_t)j * HALF + d0;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const float2 cs = __ldg(tr + e);
      // lower half: a*c - b*s with a = own, b = partner; upper half: b*c + a*s with b = own, a = partner
      kf[e] = upper ? fmaf(oth[e], cs.y, own[e] * cs.x) : fmaf(-oth[e], cs.y, own[e] * cs.x);
    }
  };

  // The new token (candidate n): its logit per head, by the warp of chunk 0.
  if (c == 0) {
    const uint4 w = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.k_new) + ((size_t)b * p.Hkv + kvh) * D + lig * EPL);
    float kf[EPL];
    rotate(w, p.n, kf);
#pragma unroll
    for (int g = 0; g < GU; ++g) {
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(qf[g][e], kf[e], s);
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      s *= p.scale2;
      if (lane == 0 && g < g_cnt) {
        p.logits[(bh0 + g) * p.ld + p.n] = s;
        p.part_ml[(bh0 + g) * p.pc + p.n_chunks] = make_float2(s, 1.f);
      }
    }
  }
  if (rows == 0) return;

  // per row group (the RPW rows of a pass) an online soft-max; the groups are merged at the end
  float m[GU], l[GU], acc[GU][EPL];
#pragma unroll
  for (int g = 0; g < GU; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
  }
  const unsigned char* k_src = static_cast<const unsigned char*>(p.K) + (((size_t)b * p.Hkv + kvh) * p.cap + row_begin) * RB;
  const unsigned char* v_src = static_cast<const unsigned char*>(p.V) + (((size_t)b * p.Hkv + kvh) * p.cap + row_begin) * RB;
#pragma unroll 4
  for (int r0 = 0; r0 < rows; r0 += RPW) {          // uniform trip count: the shuffles need the whole warp
    const int r = r0 + sub;
    const bool live = r < rows;
    const int rr = live ? r : rows - 1;
    const uint4 kw = __ldg(reinterpret_cast<const uint4*>(k_src + (size_t)rr * RB) + lig);
    const uint4 vw = __ldg(reinterpret_cast<const uint4*>(v_src + (size_t)rr * RB) + lig);
    float kf[EPL], vf[EPL];
    rotate(kw, row_begin + rr, kf);
    Vec16<T>::unpack(vw, vf);
#pragma unroll
    for (int g = 0; g < GU; ++g) {
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(qf[g][e], kf[e], s);
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      s *= p.scale2;
      if (live) {
        if (lig == 0 && g < g_cnt) p.logits[(bh0 + g) * p.ld + row_begin + r] = s;
        const float m_new = fmaxf(m[g], s);
        const float corr = exp2_diff(m[g], m_new);
        const float w = exp2f(s - m_new);
        l[g] = fmaf(l[g], corr, w);
        m[g] = m_new;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(w, vf[e], acc[g][e] * corr);
      }
    }
  }
  // merge the RPW row groups (lanes with equal lig): common maximum, rescaled sums
#pragma unroll
  for (int g = 0; g < GU; ++g) {
    float M = m[g];
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float sc = exp2_diff(m[g], M);
    float L = l[g] * sc;
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      float a = acc[g][e] * sc;
#pragma unroll
      for (int o = LPR; o < 32; o <<= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      acc[g][e] = a;
    }
    if (g < g_cnt && sub == 0) {
      float* dst = p.part_acc + ((bh0 + g) * (size_t)(p.pc - 1) + c) * D + lig * EPL;
#pragma unroll
      for (int e = 0; e < EPL; e += 4)
        *reinterpret_cast<float4*>(dst + e) = make_float4(acc[g][e], acc[g][e + 1], acc[g][e + 2], acc[g][e + 3]);
      if (lane == 0) p.part_ml[(bh0 + g) * p.pc + c] = make_float2(M, L);
    }
  }
}

}  // namespace tova
