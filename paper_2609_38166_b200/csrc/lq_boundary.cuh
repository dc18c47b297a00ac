// Window-boundary work on one 128x128 state held as 8x8 register tiles by a CTA of 256 threads:
// reconstruction of the dense state from the window representation (Eq. 7) and its quantization
// (Compensator-Token fit by power iteration on all r vectors at once, Eqs. 5-6; residual smoothing, Sec. 3.4;
// per-value-channel symmetric 8-bit codes, Appendix B.3).
#pragma once
#include "lq_common.cuh"

namespace lq {

// Shared-memory plan of the boundary kernels (in floats).  A fixed part (working vectors of the fit, the
// compensators widened to fp32) is followed by one or two staging buffers, each holding everything that is read
// from global memory for one head: with two, the next head of the CTA is fetched while this one is computed.
struct BoundarySmem {
  // fixed part
  float *ck;     // [r][128]  compensator keys widened to fp32
  float *cu;     // [r][128]  compensator values widened to fp32
  float *vec;    // [128]     row-sum results (row mean-abs)
  float *colv;   // [128]     1 / c
  float *part;   // [8][4][128] per-warp column partial sums of four vectors (column maxima: [8][128])
  float *gam;    // [128]     Gamma_{1:n}
  float *gram;   // [16][16]  Gram matrix of the vectors being orthonormalised (lower triangle), later K^T K
  float *chol;   // [16][16]  its Cholesky factor L (strictly lower triangle), then [16] 1 / L_hh, [16] alive flags
  // staging buffer `buf`
  float *kd;     // [W][128]  buffered write keys, turned in place into Gamma_{j+1:n} kt_j
  float *bu;     // [W][128]  buffered corrections u_j
  float *ba;     // [W][128]  diagonal-gate decays of the records (diagonal gate only), else [MAX_W]
  float *cs;     // [128]     smoothing scales c
  float *ss;     // [128]     code steps s_j = B_j / 127
  uint16_t *ckh; // [r][128]  compensator keys as stored (fp16 bits)
  uint16_t *cuh; // [r][128]  compensator values as stored
  uint8_t *zt;   // [128][128] codes Z^T, 16-byte chunk q of row v stored at chunk q ^ ((v >> 3) & 7)
  __half *raw;   // fp16 records only: [W] rows as stored (kt | u | (alpha)), widened into kd, bu by the decay scan
  __host__ __device__ static constexpr int fixed_floats(int r) {
    return 2 * r * D + 35 * D + 2 * MAX_R * MAX_R + 2 * MAX_R;
  }
  __host__ __device__ static constexpr int stage_floats(int W, int r, bool diag, bool rec16) {
    return 2 * W * D + (diag ? W * D : MAX_W) + 2 * D + r * D + D * D / 4 + (rec16 ? W * record_floats(diag) / 2 : 0);
  }
  __device__ __forceinline__ BoundarySmem(float *base, int W, int r, bool diag, bool rec16, int buf) {
    ck = base; cu = ck + r * D; vec = cu + r * D; colv = vec + D; part = colv + D; gam = part + 32 * D;
    gram = gam + D; chol = gram + MAX_R * MAX_R;
    kd = base + fixed_floats(r) + buf * stage_floats(W, r, diag, rec16);
    bu = kd + W * D; ba = bu + W * D; cs = ba + (diag ? W * D : MAX_W); ss = cs + D;
    ckh = reinterpret_cast<uint16_t *>(ss + D); cuh = ckh + r * D;
    zt = reinterpret_cast<uint8_t *>(cuh + r * D);
    raw = reinterpret_cast<__half *>(zt + D * D);
  }
  static size_t bytes(int W, int r, bool diag, bool rec16, int bufs) {
    return sizeof(float) * (size_t)(fixed_floats(r) + bufs * stage_floats(W, r, diag, rec16));
  }
  // two staging buffers while two CTAs with two buffers each still fit on an SM
  static int buffers(int W, int r, bool diag, bool rec16) { return bytes(W, r, diag, rec16, 2) <= 110 * 1024 ? 2 : 1; }
};

// Issue the asynchronous copies that bring head bh (its codes, scales, compensators and n records) into the
// staging buffer of sm.  The caller commits the group and later waits for it.
template <int GATE, bool R16>
__device__ __forceinline__ void stage_issue(const Params &p, const BoundarySmem &sm, const Tile &t, size_t bh, int n) {
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  constexpr int RF = record_floats(DIAG);
  const int r = p.r;
  const uint8_t *hb = p.head(bh);
  for (int e = t.tid; e < D * D / 16; e += 256) {             // codes: 1024 chunks of 16 bytes
    const int v = e >> 3, q = e & 7;
    cp_async16(sm.zt + v * D + 16 * (q ^ ((v >> 3) & 7)), hb + HB_CODES + 16 * e);
  }
  if (R16) {                                                  // the n rows are one contiguous piece of fp16 values
    const __half *rec = p.record<__half>(bh, 0, DIAG);
    for (int e = t.tid; e < n * (RF / 8); e += 256) cp_async16(sm.raw + 8 * e, rec + 8 * e);
  } else {
    const float *rec = p.record<float>(bh, 0, DIAG);
    for (int e = t.tid; e < n * (D / 4); e += 256) {
      const int j = e / (D / 4), q4 = 4 * (e % (D / 4));
      cp_async16(sm.kd + j * D + q4, rec + j * RF + REC_KT + q4);
      cp_async16(sm.bu + j * D + q4, rec + j * RF + REC_U + q4);
      if (DIAG) cp_async16(sm.ba + j * D + q4, rec + j * RF + REC_A + q4);
    }
  }
  if (!DIAG && t.tid < n) cp_async4(sm.ba + t.tid, p.decays + bh * (size_t)p.W + t.tid);
  if (t.tid < D / 4) cp_async16(sm.ss + 4 * t.tid, hb + HB_COL_SCALE + 16 * t.tid);
  else if (t.tid < D / 2) cp_async16(sm.cs + 4 * (t.tid - D / 4), hb + HB_ROW_SMOOTH + 16 * (t.tid - D / 4));
  for (int e = t.tid; e < r * D / 4; e += 256)                // 2 r rows of 256 bytes, contiguous in the head block
    cp_async16(sm.ckh + 8 * e, hb + HB_COMP_K + 16 * e);      // (cuh follows ckh in the buffer as in the block)
}

// M += x y^T on the register tile, two columns per instruction (fma.rn.f32x2 is two independent round-to-nearest
// FMAs, so the values are those of fmaf; what it halves is the issue slots of the phases that are bound by them).
__device__ __forceinline__ void rank1_update(float (&M)[8][8], const float (&x)[8], const float (&y)[8]) {
#pragma unroll
  for (int a = 0; a < 8; a++) {
    const float2 xa = make_float2(x[a], x[a]);
#pragma unroll
    for (int b = 0; b < 8; b += 2) {
      const float2 m = __ffma2_rn(xa, make_float2(y[b], y[b + 1]), make_float2(M[a][b], M[a][b + 1]));
      M[a][b] = m.x;
      M[a][b + 1] = m.y;
    }
  }
}

// Eq. 7 for the tile of thread t: M = Gamma_{1:n}[C (Z/127) B + Kc Uc^T] + sum_j Gamma_{j+1:n} kt_j u_j^T,
// evaluated per element as  base = c_i*(Z_ij*s_j) with s_j the stored code step; base = fma(kc_hi, uc_hj, base) for h = 0..r-1;
// x = gamma_i*base; x = fma(kd_ji, u_jj, x) for j = 0..n-1.  No sum crosses threads.
// Leaves the CTA's shared memory holding the records; ends after its last read of it (no trailing barrier).
template <int GATE, bool R16>
__device__ __forceinline__ void reconstruct_tile(const Params &p, const BoundarySmem &sm, const Tile &t, size_t bh,
                                                 int n, float (&M)[8][8]) {
  const int r = p.r;
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  constexpr int RF = record_floats(DIAG);
  // the staging buffer has landed and the CTA has synchronised (the caller did both)
  // cumulative decays, newest record first (Appendix B.2): kd_j = Gamma_{j+1:n} kt_j, gam = Gamma_{1:n};
  // the other half of the CTA widens the compensators meanwhile
  if (t.tid < D) {
    const int i = t.tid;
    // record j's write key and decay for channel i (fp16 records are widened here, on the way into kd)
    auto kt_at = [&](int jj) { return R16 ? __half2float(sm.raw[jj * RF + REC_KT + i]) : sm.kd[jj * D + i]; };
    auto a_at = [&](int jj) {
      return !DIAG ? sm.ba[jj] : R16 ? __half2float(sm.raw[jj * RF + REC_A + i]) : sm.ba[jj * D + i];
    };
    float g = 1.0f;
    int j = n - 1;
    for (; j >= 3; j -= 4) {                                  // four records per trip: the loads go out together
      float kt[4], a[4];
#pragma unroll
      for (int e = 0; e < 4; e++) {
        kt[e] = kt_at(j - e);
        a[e] = a_at(j - e);
      }
#pragma unroll
      for (int e = 0; e < 4; e++) {
        sm.kd[(j - e) * D + i] = g * kt[e];
        g = g * a[e];
      }
    }
    for (; j >= 0; j--) {
      sm.kd[j * D + i] = g * kt_at(j);
      g = g * a_at(j);
    }
    sm.gam[i] = g;
  } else {
    for (int e = t.tid - D; e < 2 * r * D; e += 256 - D) sm.ck[e] = f16_bits(sm.ckh[e]);   // ck and cu are adjacent
    if (R16)                                                  // fp16 records: the u rows, widened
      for (int e = t.tid - D; e < n * D; e += 256 - D) sm.bu[e] = __half2float(sm.raw[(e / D) * RF + REC_U + (e % D)]);
  }
  __syncthreads();
  LQ_BTICK(2);

  float ci[8], gi[8], sj[8];
  load8(sm.cs + 8 * t.ty, ci);
  load8(sm.gam + 8 * t.ty, gi);
  load8(sm.ss + 8 * t.tx, sj);
#pragma unroll
  for (int b = 0; b < 8; b++) {
    // column v = 8 tx + b of the tile: bytes 8 ty .. 8 ty + 7 of row v of Z^T (chunk ty / 2, swizzled by tx)
    const uint2 zz = *reinterpret_cast<const uint2 *>(sm.zt + (8 * t.tx + b) * D + 16 * ((t.ty >> 1) ^ (t.tx & 7)) +
                                                      8 * (t.ty & 1));
    // int8 -> fp32 without the conversion unit: byte + 128 placed in the low mantissa bits of 2^23, minus 2^23 + 128
    const uint32_t lo = zz.x ^ 0x80808080u, hi = zz.y ^ 0x80808080u;
#pragma unroll
    for (int a = 0; a < 8; a++) {
      const uint32_t word = a < 4 ? lo : hi;
      const float zf = __uint_as_float(__byte_perm(word, 0x4B000000u, 0x7540 | (a & 3))) - 8388736.0f;
      M[a][b] = ci[a] * (zf * sj[b]);
    }
  }
  for (int h = 0; h < r; h++) {
    float kc[8], uc[8];
    load8(sm.ck + h * D + 8 * t.ty, kc);
    load8(sm.cu + h * D + 8 * t.tx, uc);
    rank1_update(M, kc, uc);
  }
#pragma unroll
  for (int a = 0; a < 8; a++)
#pragma unroll
    for (int b = 0; b < 8; b++) M[a][b] = gi[a] * M[a][b];
  for (int j = 0; j < n; j++) {
    float kj[8], uj[8];
    load8(sm.kd + j * D + 8 * t.ty, kj);
    load8(sm.bu + j * D + 8 * t.tx, uj);
    rank1_update(M, kj, uj);
  }
  LQ_BTICK(3);
}

// ---- pieces of the Compensator-Token fit: power iteration on all r vectors at once ----

// Entry j of start vector h where no buffered record supplies one: -1 where h and j share an odd number of bits
__device__ __forceinline__ float walsh_entry(int h, int j) { return (__popc(h & j) & 1) ? -1.0f : 1.0f; }

// Lower triangle of the Gram matrix of the nv vectors X[0..nv-1] (rows of 128 floats in shared memory), one dot
// product per half-warp and trip.  Barrier before (X complete) and after (G complete) are the caller's.
__device__ __forceinline__ void gram_lower(const float *X, int nv, float *G, const Tile &t, bool with_diagonal) {
  const int hw = t.tid >> 4, c = t.lane & 15;
  const int npairs = with_diagonal ? nv * (nv + 1) / 2 : nv * (nv - 1) / 2;
  for (int base = 0; base < npairs; base += 16) {            // the same trip count for every thread of the CTA
    const int idx = base + hw;
    const int ii = idx < npairs ? idx : 0;
    int a = 0;                                               // ii = a (a + 1) / 2 + b with b <= a, without a loop
#pragma unroll
    for (int e = 1; e < MAX_R; e++) a += ii >= e * (e + 1) / 2;
    int b = ii - a * (a + 1) / 2;
    if (!with_diagonal) a += 1;                              // pairs b < a only
    const float d = dot128_shared(X + a * D, X + b * D, c);
    if (idx < npairs && c == 0) G[a * MAX_R + b] = d;
  }
}

// Cholesky factor of the Gram matrix of up to four vectors, by one thread, in registers (all loads first):
// L (strictly lower part), inv[h] = 1 / L_hh, alive[h], to shared memory.  Same arithmetic as the warp's version below.
__device__ __forceinline__ void cholesky_lower_4(const float *G, int nv, float *L) {
  float *inv = L + MAX_R * MAX_R, *alive = inv + MAX_R;
  float g[4][4], l[4][4], iv[4];
#pragma unroll
  for (int h = 0; h < 4; h++)
#pragma unroll
    for (int j = 0; j <= h; j++) g[h][j] = h < nv ? G[h * MAX_R + j] : 0.0f;
#pragma unroll
  for (int h = 0; h < 4; h++) {
#pragma unroll
    for (int j = 0; j < h; j++) {
      float sacc = g[h][j];
#pragma unroll
      for (int m = 0; m < j; m++) sacc = fmaf(-l[h][m], l[j][m], sacc);
      l[h][j] = sacc * iv[j];
    }
    float d = g[h][h];
#pragma unroll
    for (int m = 0; m < h; m++) d = fmaf(-l[h][m], l[h][m], d);
    const bool ok = g[h][h] >= 1e-30f && d > 1e-6f * g[h][h];
    iv[h] = ok ? 1.0f / sqrtf(d) : 0.0f;
    if (h < nv) {
#pragma unroll
      for (int j = 0; j < h; j++) L[h * MAX_R + j] = l[h][j];
      inv[h] = iv[h];
      alive[h] = ok ? 1.0f : 0.0f;
    }
  }
}

// Cholesky factor of the Gram matrix, by one warp: lane h owns row h of L.  Column by column: lane j finishes
// L_jj from its own row, the lanes below it their entry of column j (the entries of row j they need come by
// shuffle from lane j); the arithmetic of an entry is  s = G_hj; s = fma(-L_hm, L_jm, s) for m < j; L_hj = s / L_jj.
// Writes L (strictly lower part), inv[h] = 1 / L_hh and alive[h] to shared memory.
// A vector whose squared length is below 1e-30, or of which the vectors before it leave no more than 1e-6 of its
// squared length, is dropped: inv = 0, which makes its orthonormalised vector and all its L entries zero.
// RM: the largest number of vectors this instance is compiled for (nv <= RM <= MAX_R).
template <int RM>
__device__ __forceinline__ void cholesky_lower_warp(const float *G, int nv, float *L, int lane) {
  float *inv = L + MAX_R * MAX_R, *alive = inv + MAX_R;
  const int h = lane;
  float g[RM], l[RM];
#pragma unroll
  for (int j = 0; j < RM; j++) {
    g[j] = (h < nv && j <= h) ? G[h * MAX_R + j] : 0.0f;
    l[j] = 0.0f;
  }
  float inv_h = 0.0f;
  bool ok_h = false;
#pragma unroll
  for (int j = 0; j < RM; j++) {
    if (j < nv) {                                            // (the same for every lane)
      float d = g[j];                                        // meaningful in lane j: G_jj minus the squares of row j
#pragma unroll
      for (int m = 0; m < j; m++) d = fmaf(-l[m], l[m], d);
      const bool ok = g[j] >= 1e-30f && d > 1e-6f * g[j];
      const float iv = ok ? 1.0f / sqrtf(d) : 0.0f;
      const float inv_j = __shfl_sync(FULL, iv, j);
      if (lane == j) { inv_h = iv; ok_h = ok; }
      float sacc = g[j];                                     // meaningful in lanes h > j: G_hj
#pragma unroll
      for (int m = 0; m < j; m++) sacc = fmaf(-l[m], __shfl_sync(FULL, l[m], j), sacc);
      if (h > j) l[j] = sacc * inv_j;
    }
  }
  if (h < nv) {
#pragma unroll
    for (int j = 0; j < RM; j++)
      if (j < h) L[h * MAX_R + j] = l[j];
    inv[h] = inv_h;
    alive[h] = ok_h ? 1.0f : 0.0f;
  }
}

// Orthonormalise the nv vectors X (rows of 128 floats in shared memory) in place, in order:
// q_h = (x_h - sum_{j<h} L_hj q_j) / L_hh, one thread per element index, its nv values in registers.
// With FINAL the results are then rounded to fp16 (what is stored as compensator keys), written to comp_k of
// head bh and kept in X as the stored values.  Begins and ends with a barrier.
template <bool FINAL, int RM>
__device__ __forceinline__ void orthonormalize(const Params &p, const BoundarySmem &sm, const Tile &t, float *X,
                                               int nv, size_t bh) {
  __syncthreads();
  gram_lower(X, nv, sm.gram, t, true);
  __syncthreads();
  LQ_BTICK(7);
  if (RM <= 4) {                                             // four dependent 1/sqrt: one thread is the shortest chain
    if (t.tid == 0) cholesky_lower_4(sm.gram, nv, sm.chol);
  } else if (t.warp == 0) {
    cholesky_lower_warp<RM>(sm.gram, nv, sm.chol, t.lane);
  }
  __syncthreads();
  LQ_BTICK(8);
  if (t.tid < D) {
    const float *L = sm.chol, *inv = L + MAX_R * MAX_R, *alive = inv + MAX_R;
    const int i = t.tid;
    float x[RM];
#pragma unroll
    for (int h = 0; h < RM; h++) x[h] = h < nv ? X[h * D + i] : 0.0f;
#pragma unroll
    for (int h = 0; h < RM; h++) {
      if (h < nv) {
#pragma unroll
        for (int j = 0; j < h; j++) x[h] = fmaf(-L[h * MAX_R + j], x[j], x[h]);
        x[h] = x[h] * inv[h];
      }
    }
#pragma unroll
    for (int h = 0; h < RM; h++) {
      if (h < nv) {
        float out = x[h];
        if (FINAL) {
          const uint16_t bits = alive[h] != 0.0f ? to_f16_bits_sat(out) : static_cast<uint16_t>(0);
          p.comp_k(bh)[h * D + i] = bits;
          out = f16_bits(bits);
        }
        X[h * D + i] = out;
      }
    }
  }
  __syncthreads();
}

// T[h] = M w_h for the nv vectors w_h (two at a time), into Tm (rows of 128 floats).  `wsrc(h, w)` loads the eight
// entries of w_h for this thread's columns.  No barrier inside.
template <typename WSrc>
__device__ __forceinline__ void rows_times_vectors(const float (&M)[8][8], const Tile &t, int nv, float *Tm, WSrc wsrc) {
  for (int h0 = 0; h0 < nv; h0 += 2) {
    const bool two = h0 + 1 < nv;
    float w0[8], w1[8], pr0[8], pr1[8];
    wsrc(h0, w0);
    wsrc(two ? h0 + 1 : h0, w1);
    row_blocks(M, w0, pr0);
    row_blocks(M, w1, pr1);
    int sel;
    const float t0 = row_tree(pr0, t.lane, sel);
    const float t1 = row_tree(pr1, t.lane, sel);
    if (t.tx < 8) {
      Tm[h0 * D + 8 * t.ty + sel] = t0;
      if (two) Tm[(h0 + 1) * D + 8 * t.ty + sel] = t1;
    }
  }
}

// Out[h] = M^T x_h for the nv vectors x_h in Xm (rows of 128 floats in shared memory), four to a round of barriers.
// Column sums in the fixed order: this thread's eight rows, its neighbour in the warp (lane ^ 16), then the
// eight warps as a balanced tree.  Begins after a barrier of the caller (Xm complete); ends with a barrier.
__device__ __forceinline__ void columns_times_vectors(const float (&M)[8][8], const BoundarySmem &sm, const Tile &t,
                                                      int nv, const float *Xm, float *Out) {
  const bool up = t.lane & 16;
  for (int h0 = 0; h0 < nv; h0 += 4) {
    const int nh = nv - h0 < 4 ? nv - h0 : 4;
    if (h0 > 0) __syncthreads();                              // the previous round's partial sums have been read
    for (int hh = 0; hh < nh; hh++) {                         // first half: own rows, then the neighbour's
      float x[8], pc[8], rr[4];
      load8(Xm + (h0 + hh) * D + 8 * t.ty, x);
      col_blocks(M, x, pc);
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const float keep = up ? pc[e + 4] : pc[e], send = up ? pc[e] : pc[e + 4];
        rr[e] = keep + __shfl_xor_sync(FULL, send, 16);
      }
      *reinterpret_cast<float4 *>(sm.part + (t.warp * 4 + hh) * D + 8 * t.tx + (up ? 4 : 0)) =
          make_float4(rr[0], rr[1], rr[2], rr[3]);
    }
    __syncthreads();
    for (int idx = t.tid; idx < nh * D; idx += 256) {         // second half: the eight warps
      const int v = idx >> 7, col = idx & (D - 1);
      const float *c = sm.part + v * D + col;
      Out[(h0 + v) * D + col] =
          ((c[0] + c[4 * D]) + (c[8 * D] + c[12 * D])) + ((c[16 * D] + c[20 * D]) + (c[24 * D] + c[28 * D]));
    }
  }
  __syncthreads();
}

// Quantize the dense state held in M (destroyed) and write codes, scales and compensators of head bh.
// Uses the fixed part of shared memory (ck, cu, vec, colv, part, gram, chol); begins with a barrier so that it
// may follow any other use of it.
// Compensator Tokens (Eqs. 5-6): power iteration on all r vectors at once.  T = M W, orthonormalise, W = M^T T,
// orthonormalise, ... n_iter times, ending on the key side; column h of W starts from the value side u of the
// (h+1)-th newest of the n records in sm.bu, from a Walsh vector where there is no such record.  The keys are
// rounded to fp16; value side h is M^T k_h - sum_{a<h} u_a (k_a^T k_h) with the stored values (the least-squares
// answer for what components 0..h-1 leave), rounded to fp16 in turn; then M -= K U^T with the stored values.
// RM: the largest r this instance is compiled for (the small matrices of the fit live in registers, RM wide).
template <int RM>
__device__ __forceinline__ void quantize_tile(const Params &p, const BoundarySmem &sm, const Tile &t, size_t bh,
                                              int n, float (&M)[8][8]) {
  const int r = p.r;
  __syncthreads();
  if (r > 0) {
    float *Tm = sm.ck, *Wm = sm.cu;                           // [r][128] each; the old compensators are done with
    for (int it = 0; it < p.n_iter; it++) {
      if (it == 0) {
        rows_times_vectors(M, t, r, Tm, [&](int h, float (&w)[8]) {
          if (h < n) {
            load8(sm.bu + (n - 1 - h) * D + 8 * t.tx, w);
          } else {
#pragma unroll
            for (int b = 0; b < 8; b++) w[b] = walsh_entry(h, 8 * t.tx + b);
          }
        });
      } else {
        rows_times_vectors(M, t, r, Tm, [&](int h, float (&w)[8]) { load8(Wm + h * D + 8 * t.tx, w); });
      }
      LQ_BTICK(10);
      if (it + 1 < p.n_iter) {
        orthonormalize<false, RM>(p, sm, t, Tm, r, bh);
        columns_times_vectors(M, sm, t, r, Tm, Wm);
        orthonormalize<false, RM>(p, sm, t, Wm, r, bh);
      }
    }
    orthonormalize<true, RM>(p, sm, t, Tm, r, bh);                // Tm now holds the keys as stored
    LQ_BTICK(11);
    gram_lower(Tm, r, sm.gram, t, false);                     // k_a^T k_h, a < h, in gram[h][a]
    columns_times_vectors(M, sm, t, r, Tm, Wm);               // M^T k_h (its barriers also publish gram)
    LQ_BTICK(13);
    if (t.tid < D) {
      const float *alive = sm.chol + MAX_R * MAX_R + MAX_R;
      const int j = t.tid;
      float x[RM], uf[RM];                                    // this column's sums, then its stored values u_a
      uint16_t ub[RM];
#pragma unroll
      for (int h = 0; h < RM; h++) x[h] = h < r ? Wm[h * D + j] : 0.0f;
#pragma unroll
      for (int h = 0; h < RM; h++) {
        if (h < r) {
#pragma unroll
          for (int a = 0; a < h; a++) x[h] = fmaf(-uf[a], sm.gram[h * MAX_R + a], x[h]);
          ub[h] = alive[h] != 0.0f ? to_f16_bits_sat(x[h]) : static_cast<uint16_t>(0);
          uf[h] = f16_bits(ub[h]);
        }
      }
#pragma unroll
      for (int h = 0; h < RM; h++) {
        if (h < r) {
          p.comp_u(bh)[h * D + j] = ub[h];
          Wm[h * D + j] = uf[h];
        }
      }
    }
    __syncthreads();
    LQ_BTICK(14);
    for (int h = 0; h < r; h++) {                             // M -= k u^T with the stored values
      float kf[8], uf[8], nk[8];
      load8(Tm + h * D + 8 * t.ty, kf);
      load8(Wm + h * D + 8 * t.tx, uf);
#pragma unroll
      for (int a = 0; a < 8; a++) nk[a] = -kf[a];
      rank1_update(M, nk, uf);
    }
  }
  LQ_BTICK(4);

  // residual smoothing: c_i = max(sqrt(mean_j |R_ij|), 1e-6)
  float c[8];
  __syncthreads();   // every read of sm.vec / sm.part above is done
  if (p.smooth) {
    float pr[8];
#pragma unroll
    for (int a = 0; a < 8; a++) {                             // even and odd columns as two chains
      float even = fabsf(M[a][0]), odd = fabsf(M[a][1]);
#pragma unroll
      for (int b = 2; b < 8; b += 2) { even = even + fabsf(M[a][b]); odd = odd + fabsf(M[a][b + 1]); }
      pr[a] = even + odd;
    }
    int sel;
    const float tot = row_tree(pr, t.lane, sel);
    if (t.tx < 8) {                                           // one thread per row: c_i and 1 / c_i
      const float ci = fmaxf(sqrtf(tot / static_cast<float>(D)), 1e-6f);
      sm.vec[8 * t.ty + sel] = ci;
      sm.colv[8 * t.ty + sel] = 1.0f / ci;
    }
    __syncthreads();
    load8(sm.vec + 8 * t.ty, c);
    if (t.tx == 0) store8(p.row_smooth(bh) + 8 * t.ty, c);
    LQ_BTICK(5);
    load8(sm.colv + 8 * t.ty, c);                             // from here on c holds 1 / c_i
#pragma unroll
    for (int a = 0; a < 8; a++) {
#pragma unroll
      for (int b = 0; b < 8; b++) M[a][b] = M[a][b] * c[a];
    }
  } else {
#pragma unroll
    for (int a = 0; a < 8; a++) c[a] = 1.0f;                  // X = R / 1 = R
    if (t.tx == 0) store8(p.row_smooth(bh) + 8 * t.ty, c);
  }
  // per-value-channel scale: column maximum of |X| (exact in any order); one thread per column finishes it
  {
    float m[8];
#pragma unroll
    for (int b = 0; b < 8; b++) {
      float s = fabsf(M[0][b]);
#pragma unroll
      for (int a = 1; a < 8; a++) s = fmaxf(s, fabsf(M[a][b]));
      m[b] = fmaxf(s, __shfl_xor_sync(FULL, s, 16));
    }
    if (t.lane < 16) store8(sm.part + t.warp * D + 8 * t.tx, m);
    __syncthreads();
    const int col = threadIdx.x;
    if (col < D) {
      float amax = sm.part[col];
#pragma unroll
      for (int wv = 1; wv < 8; wv++) amax = fmaxf(amax, sm.part[wv * D + col]);
      p.col_scale(bh)[col] = amax / 127.0f;                   // stored as the step of the code, B_j / 127
      sm.cs[col] = amax > 0.0f ? 127.0f / amax : 0.0f;
    }
    __syncthreads();
  }
  LQ_BTICK(6);
  float inv[8];
  load8(sm.cs + 8 * t.tx, inv);
  int8_t *ZT = p.codes(bh);
#pragma unroll
  for (int b = 0; b < 8; b++) {
    // |X * inv| <= 127 (1 + 2^-23), so the nearest integer (ties to even) is already inside [-127, 127]
    int z[8];
#pragma unroll
    for (int a = 0; a < 8; a++) z[a] = __float_as_int(M[a][b] * inv[b] + 12582912.0f);   // + 1.5 * 2^23: the low
    // mantissa byte of the sum is the nearest integer (ties to even) in two's complement
    const uint32_t lo = __byte_perm(__byte_perm(z[0], z[1], 0x0040), __byte_perm(z[2], z[3], 0x0040), 0x5410);
    const uint32_t hi = __byte_perm(__byte_perm(z[4], z[5], 0x0040), __byte_perm(z[6], z[7], 0x0040), 0x5410);
    *reinterpret_cast<uint2 *>(ZT + (8 * t.tx + b) * D + 8 * t.ty) = make_uint2(lo, hi);
  }
}

}  // namespace lq
