// "Per-window BF16" (the -w baseline of Fig. 3 and Table 2): the window algebra of Sec. 3.2 with the boundary
// state kept as the dense state rounded to bfloat16 once per window - no scale, no smoothing, no compensators.
//
// Between boundaries a head is  S_l = Gamma_{1:l} S0 + sum_j Gamma_{j+1:l} kt_j u_j^T  (Eq. 4) with S0 in bfloat16;
// a token reads it with x = alpha (.) k and x = alpha (.) q exactly like the 8-bit path reads Eq. 7, only the
// boundary-state term is the plain binary32 product S0^T (Gamma x) in the fixed summation order.  The head block
// is S0^T, [d_v][d_k] bfloat16: the eight values a lane fetches with one 16-byte load are one block of the sum.
#pragma once
#include "lq_common.cuh"

namespace lq {

constexpr int BF16W_HEAD_BYTES = 2 * D * D;
constexpr int BF16W_CHUNK = 16;              // records whose decayed keys are held in shared memory at a time

__device__ __forceinline__ uint16_t *bf16w_state(const Params &p, size_t bh) {
  return reinterpret_cast<uint16_t *>(p.heads + bh * (size_t)BF16W_HEAD_BYTES);
}

// eight bfloat16 values as four (even, odd) pairs
__device__ __forceinline__ void widen8_bf16(const uint4 &w, float2 (&x)[4]) {
  const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int e = 0; e < 4; e++) x[e] = make_float2(__uint_as_float(ws[e] << 16), __uint_as_float(ws[e] & 0xFFFF0000u));
}

// ---------------------------------------------------------------------------------------------
// One decode token of one head per CTA of 256 threads.  Threads 0..127 own one key channel (and later one value
// channel) each; for the sums over the key index the CTA is sixteen groups of sixteen lanes, lane c holding
// block c (terms 8c..8c+7) and the groups sharing out records, then columns.  The head's buffered records are
// copied into shared memory (bf16w_decode_smem bytes, dynamic) while the state is on its way into registers, so a
// head waits for the memory system once.
// ---------------------------------------------------------------------------------------------
inline size_t bf16w_decode_smem(int W, bool diag, bool rec16) {
  return (size_t)W * record_floats(diag) * (rec16 ? 2 : 4);
}

template <int GATE, bool R16>
__global__ void __launch_bounds__(256, 4) bf16w_decode_kernel(const Params p) {
  using rec_t = typename std::conditional<R16, __half, float>::type;
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  constexpr int RF = record_floats(DIAG);
  __shared__ __align__(16) float gk_s[BF16W_CHUNK * D], gq_s[BF16W_CHUNK * D];
  __shared__ __align__(16) float kt_s[D], q_s[D], xk_s[D], xq_s[D], rk_s[D], rq_s[D];
  __shared__ float pk_s[MAX_W], pq_s[MAX_W], dec_s[MAX_W];
  __shared__ float ktq_s;
  extern __shared__ float4 lq_bf16w_rec4[];
  rec_t *rec_s = reinterpret_cast<rec_t *>(lq_bf16w_rec4);    // [n][RF], the rows as stored
  grid_dependency_wait();
  const size_t bh = blockIdx.x;
  const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);
  const int tid = threadIdx.x, c = tid & 15, G = tid >> 4;
  const int win = p.win_pos[b];              // (the last head to arrive rewrites it, after every head has read it)
  // the boundary state: column G + 16 m, block c, for m = 0..7 - all of it in flight from here on, before the
  // window position above is back
  const uint16_t *S0T = bf16w_state(p, bh);
  uint4 w[8];
#pragma unroll
  for (int m = 0; m < 8; m++) w[m] = __ldcs(reinterpret_cast<const uint4 *>(S0T + (G + 16 * m) * D + 8 * c));
  const int n = win & 0xFFFF;
  if (n >= p.W) return;                      // no room for a record: the sequence gets no token
  {
    constexpr int PER16 = 16 / sizeof(rec_t);                 // elements per 16-byte piece
    const rec_t *rows = p.record<rec_t>(bh, 0, DIAG);         // the n rows are one contiguous piece
    for (int e = tid; e < n * (RF / PER16); e += 256) cp_async16(rec_s + PER16 * e, rows + PER16 * e);
    cp_async_commit();
  }

  float k_i = 0.0f, q_i = 0.0f, kt_i = 0.0f, a_i = 0.0f, g = 0.0f;
  if (tid < D) {
    const int group = p.heads_v / p.heads_qk;
    const size_t qk_off = ((size_t)b * p.heads_qk + hv / group) * D;
    k_i = bf16_bits(p.k[qk_off + tid]);
    q_i = bf16_bits(p.q[qk_off + tid]);
    a_i = DIAG ? bf16_bits(p.alpha[bh * D + tid]) : bf16_bits(p.alpha[bh]);
    kt_i = bf16_bits(p.beta[bh]) * k_i;
    kt_s[tid] = kt_i;
    q_s[tid] = q_i;
    g = a_i;
  } else if (!DIAG && tid - D < n) {
    dec_s[tid - D] = p.decays[bh * (size_t)p.W + (tid - D)];
  }
  cp_async_wait_all();
  __syncthreads();

  // the buffered records, newest first: projections of their write keys on Gamma_{j+1:l} k and Gamma_{j+1:l} q
  for (int top = n - 1; top >= 0; top -= BF16W_CHUNK) {
    const int cnt = top + 1 < BF16W_CHUNK ? top + 1 : BF16W_CHUNK;      // records top, top-1, ..., top-cnt+1
    if (tid < D) {
#pragma unroll 4
      for (int e = 0; e < cnt; e++) {
        const int j = top - e;
        gk_s[e * D + tid] = g * k_i;
        gq_s[e * D + tid] = g * q_i;
        const float dec = DIAG ? static_cast<float>(rec_s[j * RF + REC_A + tid]) : dec_s[j];
        g = g * dec;
      }
    }
    __syncthreads();
    {
      // group G takes record top - G; a group without one repeats the chunk's last record and drops the result,
      // so that every lane of a warp takes part in the reduction
      const int e = G < cnt ? G : cnt - 1;
      const rec_t *kt_row = rec_s + (top - e) * RF + REC_KT;
      float2 a2[4], b2[4];
      load8p(kt_row + 8 * c, a2);
      load8p(gk_s + e * D + 8 * c, b2);
      const float pk = tree16(block8(a2, b2));
      load8p(gq_s + e * D + 8 * c, b2);
      const float pq = tree16(block8(a2, b2));
      if (G < cnt && c == 0) { pk_s[top - e] = pk; pq_s[top - e] = pq; }
    }
    __syncthreads();
  }
  // g = Gamma_{1:l}: what the boundary state has decayed by
  if (tid < D) { xk_s[tid] = g * k_i; xq_s[tid] = g * q_i; }
  __syncthreads();
  if (tid < 32) {
    const float ktq = dot128_shared(kt_s, q_s, c);
    if (tid == 0) ktq_s = ktq;
  }
  {
    float2 xk2[4], xq2[4];
    load8p(xk_s + 8 * c, xk2);
    load8p(xq_s + 8 * c, xq2);
#pragma unroll
    for (int m = 0; m < 8; m++) {
      float2 s2[4];
      widen8_bf16(w[m], s2);
      const float rk = tree16(block8(s2, xk2));
      const float rq = tree16(block8(s2, xq2));
      if (c == 0) { rk_s[G + 16 * m] = rk; rq_s[G + 16 * m] = rq; }
    }
  }
  __syncthreads();
  if (tid < D) {
    // the records' terms: their own sum, from the newest record back, added as one number
    float sk = 0.0f, sq = 0.0f;
#pragma unroll 4
    for (int jj = n - 1; jj >= 0; jj--) {
      const float uj = static_cast<float>(rec_s[jj * RF + REC_U + tid]);
      sk = fmaf(uj, pk_s[jj], sk);
      sq = fmaf(uj, pq_s[jj], sq);
    }
    const float rk = rk_s[tid] + sk, rq = rq_s[tid] + sq;
    const float v_j = bf16_bits(p.v[bh * D + tid]);
    const float u = p.delta ? v_j - rk : v_j;                 // Eq. 3
    p.o[bh * D + tid] = fmaf(u, ktq_s, rq);                   // S_l^T q = S_{l-1}^T (alpha.q) + u (kt^T q)
    rec_t *row = p.record<rec_t>(bh, n, DIAG);
    if (R16) {
      reinterpret_cast<uint16_t *>(row)[REC_KT + tid] = to_f16_bits_sat(kt_i);
      reinterpret_cast<uint16_t *>(row)[REC_U + tid] = to_f16_bits_sat(u);
      if (DIAG) reinterpret_cast<uint16_t *>(row)[REC_A + tid] = to_f16_bits_sat(a_i);
    } else {
      reinterpret_cast<float *>(row)[REC_KT + tid] = kt_i;
      reinterpret_cast<float *>(row)[REC_U + tid] = u;
      if (DIAG) reinterpret_cast<float *>(row)[REC_A + tid] = a_i;
    }
    if (!DIAG && tid == 0) p.decays[bh * (size_t)p.W + n] = a_i;
  }
  __syncthreads();
  if (tid == 0) arrive_and_set(p.win_pos, b, p.heads_v, n + 1);
}

// ---------------------------------------------------------------------------------------------
// Boundary: persistent CTAs of 256 threads (8x8 register tiles), each striding over the heads and taking those
// that are due.
// MODE 0: S0 <- bf16(Gamma_{1:n} S0 + sum_j Gamma_{j+1:n} kt_j u_j^T) for the sequences that are due (Eq. 4)
// MODE 1: S0 <- bf16(dense fp32 state)          MODE 2: dense fp32 state <- the sum above, nothing else changes
// Dynamic shared memory: bf16w_boundary_smem(...) bytes: the n rows as stored, then kd, u and Gamma in fp32.
// ---------------------------------------------------------------------------------------------
inline size_t bf16w_boundary_smem(int W, bool diag, bool rec16) {
  return bf16w_decode_smem(W, diag, rec16) + sizeof(float) * (size_t)(2 * W + 1) * D;
}

template <int GATE, int MODE, bool R16>
__device__ __forceinline__ void bf16w_boundary_head(const Params &p, unsigned char *smem, float *dec_s, const Tile &t,
                                                    size_t bh, int n) {
  using rec_t = typename std::conditional<R16, __half, float>::type;
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  constexpr int RF = record_floats(DIAG);
  rec_t *raw_s = reinterpret_cast<rec_t *>(smem);
  float *kd_s = reinterpret_cast<float *>(smem + (size_t)p.W * RF * sizeof(rec_t));
  float *bu_s = kd_s + p.W * D, *gam_s = bu_s + p.W * D;
  const int b = static_cast<int>(bh / p.heads_v);
  float M[8][8];
  uint16_t *S0T = bf16w_state(p, bh);
  if (MODE == 1) {
    const float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) load8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);
  } else {
    {
      constexpr int PER16 = 16 / sizeof(rec_t);
      const rec_t *rows = p.record<rec_t>(bh, 0, DIAG);       // the n rows are one contiguous piece
      for (int e = t.tid; e < n * (RF / PER16); e += 256) cp_async16(raw_s + PER16 * e, rows + PER16 * e);
      cp_async_commit();
    }
    uint4 wv[8];                                              // column 8tx+bcol, rows 8ty..8ty+7
#pragma unroll
    for (int bcol = 0; bcol < 8; bcol++)
      wv[bcol] = *reinterpret_cast<const uint4 *>(S0T + (8 * t.tx + bcol) * D + 8 * t.ty);
    if (!DIAG && t.tid < n) dec_s[t.tid] = p.decays[bh * (size_t)p.W + t.tid];
    cp_async_wait_all();
    __syncthreads();
    // cumulative decays, newest record first (Appendix B.2): kd_j = Gamma_{j+1:n} kt_j, gam = Gamma_{1:n}
    if (t.tid < D) {
      float gam = 1.0f;
      for (int j = n - 1; j >= 0; j--) {
        kd_s[j * D + t.tid] = gam * static_cast<float>(raw_s[j * RF + REC_KT + t.tid]);
        const float dec = DIAG ? static_cast<float>(raw_s[j * RF + REC_A + t.tid]) : dec_s[j];
        gam = gam * dec;
      }
      gam_s[t.tid] = gam;
    } else {
      const int i = t.tid - D;
      for (int j = 0; j < n; j++) bu_s[j * D + i] = static_cast<float>(raw_s[j * RF + REC_U + i]);
    }
#pragma unroll
    for (int bcol = 0; bcol < 8; bcol++) {
      float2 s2[4];
      widen8_bf16(wv[bcol], s2);
#pragma unroll
      for (int e = 0; e < 4; e++) { M[2 * e][bcol] = s2[e].x; M[2 * e + 1][bcol] = s2[e].y; }
    }
    __syncthreads();
    float gi[8];
    load8(gam_s + 8 * t.ty, gi);
#pragma unroll
    for (int a = 0; a < 8; a++)
#pragma unroll
      for (int bcol = 0; bcol < 8; bcol++) M[a][bcol] = gi[a] * M[a][bcol];
    for (int j = 0; j < n; j++) {                             // oldest record first
      float kj[8], uj[8];
      load8(kd_s + j * D + 8 * t.ty, kj);
      load8(bu_s + j * D + 8 * t.tx, uj);
#pragma unroll
      for (int a = 0; a < 8; a++)
#pragma unroll
        for (int bcol = 0; bcol < 8; bcol++) M[a][bcol] = fmaf(kj[a], uj[bcol], M[a][bcol]);
    }
  }
  if (MODE == 2) {
    float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) store8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);
  } else {
#pragma unroll
    for (int bcol = 0; bcol < 8; bcol++) {
      uint32_t ws[4];
#pragma unroll
      for (int e = 0; e < 4; e++)
        ws[e] = (uint32_t)to_bf16_bits(M[2 * e][bcol]) | ((uint32_t)to_bf16_bits(M[2 * e + 1][bcol]) << 16);
      *reinterpret_cast<uint4 *>(S0T + (8 * t.tx + bcol) * D + 8 * t.ty) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
    }
    __syncthreads();
    if (t.tid == 0) {
      if (MODE == 0) arrive_and_set(p.win_pos, b, p.heads_v, 0);
      else p.win_pos[b] = 0;                 // nobody reads win_pos in this mode
    }
  }
}

template <int GATE, int MODE, bool R16>
__global__ void __launch_bounds__(256, 2) bf16w_boundary_kernel(const Params p) {
  extern __shared__ float4 lq_bf16w_smem4[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(lq_bf16w_smem4);
  __shared__ uint32_t todo_mask;
  __shared__ int todo_n[32];
  __shared__ float dec_s[MAX_W];
  const Tile t;
  const size_t nh = (size_t)p.batch * p.heads_v;
  grid_dependency_wait();
  // The CTA owns heads blockIdx.x + k * gridDim.x; warp 0 looks at 32 of them at a time (one load each, all in
  // flight together) and publishes which are due and how many records each holds.
  for (size_t base = blockIdx.x; base < nh; base += 32 * (size_t)gridDim.x) {
    if (t.warp == 0) {
      const size_t cand = base + t.lane * (size_t)gridDim.x;
      bool want = false;
      int n_mine = 0;
      if (cand < nh) {
        if (MODE != 1) n_mine = p.win_pos[cand / p.heads_v] & 0xFFFF;
        want = MODE != 0 || n_mine == p.W || (p.force && n_mine > 0);
      }
      const uint32_t m = __ballot_sync(FULL, want);
      todo_n[t.lane] = n_mine > p.W ? p.W : n_mine;
      if (t.lane == 0) todo_mask = m;
    }
    __syncthreads();
    uint32_t mask = todo_mask;
    while (mask) {
      const int kbit = __ffs(mask) - 1;
      mask &= mask - 1;
      bf16w_boundary_head<GATE, MODE, R16>(p, smem, dec_s, t, base + kbit * (size_t)gridDim.x, todo_n[kbit]);
      __syncthreads();                       // this head's use of shared memory is over
    }
    __syncthreads();                         // todo_mask / todo_n are rewritten by the next round
  }
}

}  // namespace lq
