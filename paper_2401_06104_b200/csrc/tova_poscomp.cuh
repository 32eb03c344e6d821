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
//   tova_poscomp_kernel     per sequence: the candidates sorted by position (bitonic
//                           sort in shared memory), the chain of compressed positions
//                           (in double, prefix sums in position order), a (cos, sin)
//                           table per candidate and frequency (angles reduced in
//                           double, fp32 from there), and the rotated query in fp32;
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
constexpr int ROPE_UNIT_HEADS = 4;     // query heads one warp of the rotating streaming kernel carries at most
// ... and for a group of G heads: 1, 2 or 4 (a warp carrying fewer heads than its template holds would repeat work)
__host__ __device__ inline int rope_unit_heads(int G) { return G >= 3 ? 4 : (G == 2 ? 2 : 1); }

struct PosCompParams {
  float2* table;      // [B,cap+1,D/2] (cos, sin) of candidate j (slot order, the new token at index n) and frequency d
  float* q_rot;       // [B,H,D] the query after rotary embedding at the new token's compressed position
  double* cpos;       // [B,cap+1] compressed positions (kept for inspection)
  double rope_base;
  double inv_freq[64];   // rope_base^(-2d/D) for d < D/2 (head_dim <= 128), computed once on the host
};

__device__ __forceinline__ double compress_gap(int g) { return (g <= 10) ? (double)g : log(log((double)g)); }

// (cos, sin) of a non-negative angle given in double, to fp32 accuracy: the angle is reduced to [-pi/4, pi/4] in
// double (x - k * pi/2; with k < 2^20 the one-term reduction is exact to ~1e-10), the remainder goes through the
// fp32 routine, and the quadrant k mod 4 picks the signs.  A sixth of the cost of the double-precision routine.
__device__ __forceinline__ float2 cos_sin_f32(double x) {
  const double k = rint(x * 0.63661977236758134308);           // 2 / pi
  const float r = (float)fma(-k, 1.57079632679489661923, x);   // pi / 2
  float sr, cr;
  sincosf(r, &sr, &cr);
  const int q = (int)((long long)k & 3);
  const float c = (q & 1) ? sr : cr, s2 = (q & 1) ? cr : sr;
  // q = 0: (c, s); 1: (-s, c); 2: (-c, -s); 3: (s, -c)
  return make_float2((q == 1 || q == 2) ? -c : c, (q >= 2) ? -s2 : s2);
}

__host__ __device__ inline int poscomp_sort_size(int cap) {   // the smallest power of two >= 32 that holds cap + 1 keys
  int n = 32;
  while (n < cap + 1) n <<= 1;
  return n;
}

// grid = (B, blocks per sequence), block = POSCOMP_THREADS.  Dynamic shared memory (poscomp_smem_bytes): the sort
// keys (64 bits each, a power of two of them), per candidate a double (the chain) and an int (its rank), plus D/2
// doubles (inverse frequencies).
__host__ __device__ inline size_t poscomp_smem_bytes(int cap, int D) {
  return sizeof(unsigned long long) * (size_t)poscomp_sort_size(cap) + sizeof(double) * ((size_t)cap + 1 + D / 2) +
         sizeof(int32_t) * ((size_t)cap + 1);
}
template <typename T, int D>
__global__ void __launch_bounds__(POSCOMP_THREADS) tova_poscomp_kernel(const StepParams p, const PosCompParams pc) {
  constexpr int NT = POSCOMP_THREADS, HALF = D / 2;
  extern __shared__ __align__(16) unsigned char pcs_raw[];
  const int b = blockIdx.x, tid = threadIdx.x;
  const int m = p.n + 1;                                   // candidates: the live rows, then the new token
  const int N = poscomp_sort_size(p.cap);
  unsigned long long* key = reinterpret_cast<unsigned long long*>(pcs_raw);   // [N] (position, candidate), sorted below
  double* chain = reinterpret_cast<double*>(key + N);      // [m] compressed position by rank
  double* inv_freq = chain + m;                            // [HALF]
  int32_t* rank = reinterpret_cast<int32_t*>(inv_freq + HALF);   // [m] rank of the candidate in position order
  const int pos_t = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;    // the streaming kernel of this step updates cur_pos later

  // Candidates in position order (equal positions, which a caller could pass, in candidate order): a bitonic sort
  // of (position, candidate) keys in shared memory, padded with keys beyond every position.
  for (int j = tid; j < N; j += NT) {
    const int pj = (j < p.n) ? p.pos[(size_t)b * p.cap + j] : pos_t;
    key[j] = (j < m) ? (((unsigned long long)(unsigned int)pj << 32) | (unsigned int)j) : ~0ull;
  }
  for (int d = tid; d < HALF; d += NT) inv_freq[d] = pc.inv_freq[d];
  __syncthreads();
  for (int k = 2; k <= N; k <<= 1) {
    // partners 32 or more apart: through shared memory, one pair per thread and turn
    for (int j = k >> 1; j >= 32; j >>= 1) {
      for (int u = tid; u < N / 2; u += NT) {
        const int t = ((u & ~(j - 1)) << 1) | (u & (j - 1));   // the pair's lower index: bit j clear
        const unsigned long long a = key[t], c = key[t | j];
        if (((t & k) == 0) ? (a > c) : (a < c)) { key[t] = c; key[t | j] = a; }
      }
      __syncthreads();
    }
    // partners inside a warp's 32 consecutive keys: in registers, by shuffle
    for (int t = tid; t < N; t += NT) {                        // N is a multiple of 32: whole warps
      unsigned long long v = key[t];
      const bool up = (t & k) == 0;
      for (int j = min(k >> 1, 16); j > 0; j >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, v, j);
        const bool lower = (t & j) == 0;
        v = (lower == up) ? (v < o ? v : o) : (v > o ? v : o);
      }
      key[t] = v;
    }
    __syncthreads();
  }
  // rank of every candidate, then the compressed gap to the predecessor in position order
  for (int r = tid; r < m; r += NT) {
    rank[(int)(key[r] & 0xffffffffu)] = r;
    chain[r] = (r > 0) ? compress_gap((int)(key[r] >> 32) - (int)(key[r - 1] >> 32)) : 0.0;
  }
  __syncthreads();
  if (tid < 32) {
    // The chain: prefix sums in position order, in double.  Every lane sums a run of consecutive ranks, the
    // runs' totals are scanned across the warp, then every lane writes its run's prefixes.
    const int per = (m + 31) / 32, r_lo = min(tid * per, m), r_hi = min(r_lo + per, m);
    double run = 0.0;
    for (int r = r_lo; r < r_hi; ++r) run += chain[r];
    double incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, incl, o);
      if (tid >= o) incl += up;
    }
    double acc = incl - run;                               // total of the runs before this lane's
    for (int r = r_lo; r < r_hi; ++r) {
      acc += chain[r];
      chain[r] = acc;
    }
  }
  __syncthreads();
  // table of (cos, sin) by candidate: the blocks of a sequence (gridDim.y of them, each having rebuilt the chain
  // for itself) take the table's entries in turn; block 0 also stores the compressed positions and the query
  float2* tab = pc.table + (size_t)b * (p.cap + 1) * HALF;
  for (int i = blockIdx.y * NT + tid; i < m * HALF; i += NT * gridDim.y) {
    const int j = i / HALF, d = i % HALF;
    tab[i] = cos_sin_f32(chain[rank[j]] * inv_freq[d]);
  }
  if (blockIdx.y != 0) return;
  for (int j = tid; j < m; j += NT) pc.cpos[(size_t)b * (p.cap + 1) + j] = chain[rank[j]];
  // the query, rotated at the new token's position (fp32)
  const double pq = chain[rank[p.n]];
  for (int i = tid; i < p.H * HALF; i += NT) {
    const int h = i / HALF, d = i % HALF;
    const float2 cs = cos_sin_f32(pq * inv_freq[d]);
    const float cf = cs.x, sf = cs.y;
    const T* qh = static_cast<const T*>(p.q) + ((size_t)b * p.H + h) * D;
    const float a = (float)qh[d], bb = (float)qh[d + HALF];
    float* dst = pc.q_rot + ((size_t)b * p.H + h) * D;
    dst[d] = a * cf - bb * sf;
    dst[d + HALF] = bb * cf + a * sf;
  }
}

// grid = (max(n_chunks,1), Hkv*hgroups, B), block = one warp.  hgroups = ceil(G / GU), GU = rope_unit_heads(G).
template <typename T, int D, int GU>
__global__ void __launch_bounds__(32) tova_split_rope_kernel(const StepParams p, const PosCompParams pc) {
  static_assert(GU == 1 || GU == 2 || GU == 4, "heads per warp");
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
    const float4* tr = reinterpret_cast<const float4*>(tab + (size_t)j * HALF + d0);   // EPL is even, rows are 16-byte aligned
#pragma unroll
    for (int e = 0; e < EPL; e += 2) {
      const float4 cs = __ldg(tr + e / 2);                  // (cos, sin) of two neighbouring frequencies
      // lower half: a*c - b*s with a = own, b = partner; upper half: b*c + a*s with b = own, a = partner
      kf[e] = upper ? fmaf(oth[e], cs.y, own[e] * cs.x) : fmaf(-oth[e], cs.y, own[e] * cs.x);
      kf[e + 1] = upper ? fmaf(oth[e + 1], cs.w, own[e + 1] * cs.z) : fmaf(-oth[e + 1], cs.w, own[e + 1] * cs.z);
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
  // One head per warp: a pass is a short chain of dependent steps (rotation, reduction over the row's lanes,
  // soft-max update) that cannot hide a trip to DRAM, so the rows of the next two passes are requested before the
  // current one is worked on.  With more heads per warp a pass is long enough, and the registers are better spent
  // on keeping more warps resident (measured: the look-ahead costs 30 % there).
  constexpr int AHEAD = (GU == 1) ? 2 : 0;
  uint4 kq[AHEAD + 1], vq[AHEAD + 1];
#pragma unroll
  for (int a = 0; a < AHEAD; ++a) {
    const int rr = min(a * RPW + sub, rows - 1);
    kq[a] = __ldg(reinterpret_cast<const uint4*>(k_src + (size_t)rr * RB) + lig);
    vq[a] = __ldg(reinterpret_cast<const uint4*>(v_src + (size_t)rr * RB) + lig);
  }
#pragma unroll(AHEAD > 0 ? 2 : 4)
  for (int r0 = 0; r0 < rows; r0 += RPW) {          // uniform trip count: the shuffles need the whole warp
    const int r = r0 + sub;
    const bool live = r < rows;
    const int rr = live ? r : rows - 1;
    {
      const int rn = min(r0 + AHEAD * RPW + sub, rows - 1);   // AHEAD = 0: this pass's own rows
      kq[AHEAD] = __ldg(reinterpret_cast<const uint4*>(k_src + (size_t)rn * RB) + lig);
      vq[AHEAD] = __ldg(reinterpret_cast<const uint4*>(v_src + (size_t)rn * RB) + lig);
    }
    const uint4 kw = kq[0], vw = vq[0];
#pragma unroll
    for (int a = 0; a < AHEAD; ++a) { kq[a] = kq[a + 1]; vq[a] = vq[a + 1]; }
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
