// Window-boundary work on one 128x128 state held as 8x8 register tiles by a CTA of 256 threads:
// reconstruction of the dense state from the window representation (Eq. 7) and its quantization
// (Compensator-Token fit by power iteration with deflation, Eqs. 5-6; residual smoothing, Sec. 3.4;
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
  float *vec;    // [128]     row-sum results (t of the power iteration, row mean-abs)
  float *colv;   // [128]     column-sum results
  float *part;   // [8][128]  per-warp column partial sums
  float *gam;    // [128]     Gamma_{1:n}
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
  __host__ __device__ static constexpr int fixed_floats(int r) { return 2 * r * D + 11 * D; }
  __host__ __device__ static constexpr int stage_floats(int W, int r, bool diag, bool rec16) {
    return 2 * W * D + (diag ? W * D : MAX_W) + 2 * D + r * D + D * D / 4 + (rec16 ? W * record_floats(diag) / 2 : 0);
  }
  __device__ __forceinline__ BoundarySmem(float *base, int W, int r, bool diag, bool rec16, int buf) {
    ck = base; cu = ck + r * D; vec = cu + r * D; colv = vec + D; part = colv + D; gam = part + 8 * D;
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

// Quantize the dense state held in M (destroyed) and write codes, scales and compensators of head bh.
// Uses sm.vec and sm.part; begins with a barrier so that it may follow any other use of shared memory.
// The power iteration of compensator h starts from the value side u of the (h+1)-th newest of the n records in
// sm.bu, scaled to unit length; from the all-equal unit vector where there is no such record or it is zero.
__device__ __forceinline__ void quantize_tile(const Params &p, const BoundarySmem &sm, const Tile &t, size_t bh,
                                              int n, float (&M)[8][8]) {
  const int r = p.r;
  __syncthreads();
  // The scales 1 / |u| of all start vectors at once, one per group of sixteen lanes (they depend on the records
  // only; taken one by one inside the loop each would cost a reduction and a reciprocal square root of latency).
  // 0 marks "no such record, or a zero one": start from the all-equal vector.  Kept in sm.gam, which is free now.
  float *start_scale = sm.gam;
  {
    // (every thread takes part in the warp-wide reduction, whatever r and n: groups without a record of
    // their own reduce record 0 and drop the result)
    const int g16 = t.tid >> 4;                               // r <= 16 = the number of groups
    const bool mine = g16 < r && g16 < n;
    const float *u = sm.bu + (mine ? n - 1 - g16 : 0) * D;
    const float nu0 = dot128_shared(u, u, t.lane & 15);
    const float s0 = mine && nu0 >= 1e-30f ? 1.0f / sqrtf(nu0) : 0.0f;
    if (g16 < r && (t.lane & 15) == 0) start_scale[g16] = s0;
  }
  __syncthreads();
  int h = 0;
  for (; h < r; h++) {
    float w[8], tn[8];
    const float w0 = 1.0f / sqrtf(static_cast<float>(D));
#pragma unroll
    for (int b = 0; b < 8; b++) w[b] = w0;
    {
      const float s0 = start_scale[h];
      if (s0 != 0.0f) {
        load8(sm.bu + (n - 1 - h) * D + 8 * t.tx, w);
#pragma unroll
        for (int b = 0; b < 8; b++) w[b] = w[b] * s0;
      }
    }
    bool vanished = false;
    for (int it = 0; it < p.n_iter; it++) {
      float pr[8];
      row_blocks(M, w, pr);                                   // t = M w
      int sel;
      const float tv = row_tree(pr, t.lane, sel);
      if (t.tx < 8) sm.vec[8 * t.ty + sel] = tv;
      __syncthreads();
      const float nu = dot128_shared(sm.vec, sm.vec, t.lane & 15);
      if (nu < 1e-30f) { vanished = true; break; }            // same value in every thread
      const float rinv = 1.0f / sqrtf(nu);
      load8(sm.vec + 8 * t.ty, tn);
#pragma unroll
      for (int a = 0; a < 8; a++) tn[a] = tn[a] * rinv;
      if (it + 1 < p.n_iter) {
        float pc[8];
        col_blocks(M, tn, pc);                                // w = M^T t
        col_tree(pc, sm.part, sm.colv, t, w);
      }
    }
    if (vanished) break;
    // store the key side in fp16 and continue with the stored values
    float kf[8], uf[8];
    uint16_t kb[8], ub[8];
#pragma unroll
    for (int a = 0; a < 8; a++) { kb[a] = to_f16_bits_sat(tn[a]); kf[a] = f16_bits(kb[a]); }
    {
      float pc[8], uraw[8];
      col_blocks(M, kf, pc);                                  // value side = M^T k
      col_tree(pc, sm.part, sm.colv, t, uraw);
#pragma unroll
      for (int b = 0; b < 8; b++) { ub[b] = to_f16_bits_sat(uraw[b]); uf[b] = f16_bits(ub[b]); }
    }
    if (t.tx == 0) {
      uint4 pk = make_uint4(kb[0] | (uint32_t)kb[1] << 16, kb[2] | (uint32_t)kb[3] << 16, kb[4] | (uint32_t)kb[5] << 16,
                            kb[6] | (uint32_t)kb[7] << 16);
      *reinterpret_cast<uint4 *>(p.comp_k(bh) + h * D + 8 * t.ty) = pk;
    }
    if (t.ty == 0) {
      uint4 pu = make_uint4(ub[0] | (uint32_t)ub[1] << 16, ub[2] | (uint32_t)ub[3] << 16, ub[4] | (uint32_t)ub[5] << 16,
                            ub[6] | (uint32_t)ub[7] << 16);
      *reinterpret_cast<uint4 *>(p.comp_u(bh) + h * D + 8 * t.tx) = pu;
    }
    float nk[8];
#pragma unroll
    for (int a = 0; a < 8; a++) nk[a] = -kf[a];
    rank1_update(M, nk, uf);                                  // M -= k u^T with the stored values
  }
  LQ_BTICK(4);
  // a vanished component means nothing is left to fit: this and all later compensators are zero
  for (; h < r; h++) {
    if (t.tx == 0) *reinterpret_cast<uint4 *>(p.comp_k(bh) + h * D + 8 * t.ty) = make_uint4(0, 0, 0, 0);
    if (t.ty == 0) *reinterpret_cast<uint4 *>(p.comp_u(bh) + h * D + 8 * t.tx) = make_uint4(0, 0, 0, 0);
  }

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
