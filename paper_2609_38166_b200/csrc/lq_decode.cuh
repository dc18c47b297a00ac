// Decode: one token for one (sequence, value head), done by a team of 128 threads (4 warps).
//
// Eq. 10 (readout of the smoothed, compensated window representation) evaluated for x = alpha.k and
// x = alpha.q in one pass over the 8-bit codes:
//   S_{l-1}^T (alpha.x) = (B/127) Z^T (C Gamma_{1:l} x) + Uc (Kc^T Gamma_{1:l} x) + sum_j u_j (kt_j^T Gamma_{j+1:l} x)
// then u = v - S_{l-1}^T(alpha.k) (Eq. 3), o = S_{l-1}^T(alpha.q) + u (kt^T q), and the record is appended.
//
// The first term is a dense int8 contraction, Z^T [128 x 128] against the two vectors.  The vectors are
// put on a 30-bit block fixed-point grid and split into four signed base-256 digits each, which gives an
// int8 operand of 128 x 8; the tensor cores (mma.sync m16n8k32, s8 x s8 -> s32) then produce exact
// integer sums, which are recombined in 64-bit integers and rounded to fp32 once.  The result does not
// depend on the order of accumulation.  The codes are stored value-channel major (Z^T, [d_v][d_k]), so
// that the key index, the contraction index, is contiguous in memory as the MMA operand layout needs.
//
// All 16 KiB of codes of a head are requested by eight 16-byte loads per thread at entry and consumed
// after the (much smaller) record walk, so a team has its whole state in flight at once.
#pragma once
#include "lq_common.cuh"

namespace lq {

struct DecodeSmem {
  float *bk, *bu, *ba;      // staged records: [W][128], [W][128], [W][128] (diag) or [MAX_W] (scalar)
  float *ck, *cu;           // compensators widened to fp32: [r][128] each
  float *kf, *qf, *kt;      // token vectors
  float *gk, *gq;           // Gamma_{1:l} k, Gamma_{1:l} q
  float *yk, *yq;           // exact integer sums of the state stream, rounded to fp32
  float *pk, *pq;           // [MAX_W + MAX_R + 1] projections; the last used slot of pq holds kt^T q
  float *gs;                // [MAX_W] scalar-gate decays Gamma_{j+1:l}
  float *wmax;              // [4 warps][2] per-warp maxima of |C Gamma k|, |C Gamma q|
  int8_t *digits;           // [8][128] digit planes: plane 4v+d = digit d of vector v (0: k, 1: q)
  __device__ __forceinline__ DecodeSmem(float *base, int W, int r, bool diag) {
    bk = base; bu = bk + W * D; ba = bu + W * D; ck = ba + (diag ? W * D : MAX_W); cu = ck + r * D;
    kf = cu + r * D; qf = kf + D; kt = qf + D; gk = kt + D; gq = gk + D; yk = gq + D; yq = yk + D;
    pk = yq + D; pq = pk + (MAX_W + MAX_R + 16); gs = pq + (MAX_W + MAX_R + 16); wmax = gs + MAX_W;
    digits = reinterpret_cast<int8_t *>(wmax + 8);
  }
  static size_t bytes(int W, int r, bool diag) {
    return sizeof(float) * (size_t)(2 * W * D + (diag ? W * D : MAX_W) + 2 * r * D + 7 * D +
                                    2 * (MAX_W + MAX_R + 16) + MAX_W + 8) + 8 * D;
  }
};

// D(16x8, s32) += A(16x32, s8, row-major) * B(32x8, s8, column-major)
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Block fixed point of a 128-vector whose largest magnitude is xmax: scale = 2^(29-e), back = 2^(e-29) with
// 2^e <= xmax < 2^(e+1); both zero when xmax < 2^-96 (the vector then counts as zero).
__device__ __forceinline__ void fixed_point_scales(float xmax, float &scale, float &back) {
  if (!(xmax >= 0x1p-96f)) { scale = 0.0f; back = 0.0f; return; }
  const int e = static_cast<int>((__float_as_uint(xmax) >> 23) & 0xFF) - 127;
  scale = __uint_as_float(static_cast<uint32_t>(29 - e + 127) << 23);
  back = __uint_as_float(static_cast<uint32_t>(e - 29 + 127) << 23);
}

// X = d0 + 256 d1 + 65536 d2 + 2^24 d3 with every digit in [-128, 127] (|X| <= 2^30)
__device__ __forceinline__ void store_digits(int X, int8_t *plane0, int i) {
#pragma unroll
  for (int d = 0; d < 4; d++) {
    const int dig = (X << 24) >> 24;      // sign-extended low byte
    plane0[d * D + i] = static_cast<int8_t>(dig);
    X = (X - dig) >> 8;
  }
}

// The work of one team on head bh; tid in [0,128) is the thread's index within the team and `bar` the id
// of the named barrier the team synchronises on (all 128 threads of the team must call this function).
template <int GATE>
__device__ __forceinline__ void decode_head(const Params &p, const DecodeSmem &sm, const size_t bh, const int tid,
                                            const int bar, const int n) {
  const int W = p.W, r = p.r;
  const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);
  auto team_sync = [&]() { asm volatile("bar.sync %0, 128;\n" ::"r"(bar) : "memory"); };

  // (1) the codes.  Warp w owns value channels 32w..32w+31 as two 16-row MMA tiles; a thread's 16 bytes of
  // a row hold the key channels 64p+16t..64p+16t+15, which serve as the A fragments of two k-blocks.
  uint4 zlo[2][2], zhi[2][2];
  {
    const int8_t *ZT = p.codes + bh * (size_t)(D * D);
#pragma unroll
    for (int mt = 0; mt < 2; mt++)
#pragma unroll
      for (int pp = 0; pp < 2; pp++) {
        const int j = 32 * warp + 16 * mt + g;
        zlo[mt][pp] = *reinterpret_cast<const uint4 *>(ZT + j * D + 64 * pp + 16 * t);
        zhi[mt][pp] = *reinterpret_cast<const uint4 *>(ZT + (j + 8) * D + 64 * pp + 16 * t);
      }
  }

  // (2) records of the window so far -> shared memory, asynchronously
  {
    const float *bk = p.buf_k + bh * (size_t)(W * D), *bu = p.buf_u + bh * (size_t)(W * D);
    for (int e = tid; e < n * (D / 4); e += 128) {
      cp_async16(sm.bk + 4 * e, bk + 4 * e);
      cp_async16(sm.bu + 4 * e, bu + 4 * e);
    }
    if (GATE == LQ_GATE_DIAG) {
      const float *ba = p.buf_a + bh * (size_t)(W * D);
      for (int e = tid; e < n * (D / 4); e += 128) cp_async16(sm.ba + 4 * e, ba + 4 * e);
    } else if (tid < n) {
      sm.ba[tid] = p.buf_a[bh * (size_t)W + tid];
    }
    cp_async_commit();
  }

  // (3) the token: thread i holds key channel i and value channel i
  const int group = p.heads_v / p.heads_qk;
  const size_t qk_off = ((size_t)b * p.heads_qk + hv / group) * D;
  const float k_i = bf16_bits(p.k[qk_off + tid]), q_i = bf16_bits(p.q[qk_off + tid]);
  const float v_j = bf16_bits(p.v[bh * D + tid]);
  const float beta = bf16_bits(p.beta[bh]);
  const float a_i = GATE == LQ_GATE_DIAG ? bf16_bits(p.alpha[bh * D + tid]) : bf16_bits(p.alpha[bh]);
  const float kt_i = beta * k_i;
  const float c_i = p.row_smooth[bh * D + tid];
  const float s_j = p.col_scale[bh * D + tid] / 127.0f;
  sm.kf[tid] = k_i; sm.qf[tid] = q_i; sm.kt[tid] = kt_i;
  {
    const uint16_t *gk = p.comp_k + bh * (size_t)(r * D), *gu = p.comp_u + bh * (size_t)(r * D);
    for (int h = 0; h < r; h++) {
      sm.ck[h * D + tid] = f16_bits(gk[h * D + tid]);
      sm.cu[h * D + tid] = f16_bits(gu[h * D + tid]);
    }
  }
  cp_async_wait_all();
  team_sync();

  // (4) cumulative decays from the newest record back (Appendix B.2).  After the loop gam = Gamma_{1:l}.
  float gam = a_i;
  if (GATE == LQ_GATE_DIAG) {
    for (int j = n - 1; j >= 0; j--) {
      const float aj = sm.ba[j * D + tid];
      sm.ba[j * D + tid] = gam;            // Gamma_{j+1:l} for channel i, in place of the record's decay
      gam = gam * aj;
    }
  } else {
    for (int j = n - 1; j >= 0; j--) {     // every thread runs the same scalar chain
      if (tid == 0) sm.gs[j] = gam;
      gam = gam * sm.ba[j];
    }
  }
  const float gk_i = gam * k_i, gq_i = gam * q_i;
  const float xk_i = c_i * gk_i, xq_i = c_i * gq_i;
  sm.gk[tid] = gk_i; sm.gq[tid] = gq_i;
  {
    float mk = fabsf(xk_i), mq = fabsf(xq_i);
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) {
      mk = fmaxf(mk, __shfl_xor_sync(FULL, mk, m));
      mq = fmaxf(mq, __shfl_xor_sync(FULL, mq, m));
    }
    if (lane == 0) { sm.wmax[2 * warp] = mk; sm.wmax[2 * warp + 1] = mq; }
  }
  team_sync();

  // (4b) the two vectors on their fixed-point grids, as digit planes for the B operand
  float back_k, back_q;
  {
    const float xmk = fmaxf(fmaxf(sm.wmax[0], sm.wmax[2]), fmaxf(sm.wmax[4], sm.wmax[6]));
    const float xmq = fmaxf(fmaxf(sm.wmax[1], sm.wmax[3]), fmaxf(sm.wmax[5], sm.wmax[7]));
    float scale_k, scale_q;
    fixed_point_scales(xmk, scale_k, back_k);
    fixed_point_scales(xmq, scale_q, back_q);
    store_digits(__float2int_rn(xk_i * scale_k), sm.digits, tid);
    store_digits(__float2int_rn(xq_i * scale_q), sm.digits + 4 * D, tid);
  }

  // (5) projections: one dot product pair per group of sixteen lanes (lane c owns block c of eight terms).
  // The trip count is the same for both halves of a warp (the shuffles of tree16 name all 32 lanes): a
  // half without a dot product of its own recomputes the last one and does not store it.
  {
    const int c = tid & 15, total = n + r + 1;
    for (int jb = 2 * warp; jb < total; jb += 8) {
      const int jown = jb + (lane >> 4);
      const int j = jown < total ? jown : total - 1;
      float a8[8], bk8[8], bq8[8];
      if (j < n) {
        load8(sm.bk + j * D + 8 * c, a8);
        float k8[8], q8[8];
        load8(sm.kf + 8 * c, k8);
        load8(sm.qf + 8 * c, q8);
        if (GATE == LQ_GATE_DIAG) {
          float g8[8];
          load8(sm.ba + j * D + 8 * c, g8);
#pragma unroll
          for (int e = 0; e < 8; e++) { bk8[e] = g8[e] * k8[e]; bq8[e] = g8[e] * q8[e]; }
        } else {
          const float gj = sm.gs[j];
#pragma unroll
          for (int e = 0; e < 8; e++) { bk8[e] = gj * k8[e]; bq8[e] = gj * q8[e]; }
        }
      } else if (j < n + r) {
        load8(sm.ck + (j - n) * D + 8 * c, a8);
        load8(sm.gk + 8 * c, bk8);
        load8(sm.gq + 8 * c, bq8);
      } else {                               // kt^T q, stored in the pq slot; the pk slot is unused
        load8(sm.kt + 8 * c, a8);
        load8(sm.qf + 8 * c, bq8);
#pragma unroll
        for (int e = 0; e < 8; e++) bk8[e] = bq8[e];
      }
      float sk = a8[0] * bk8[0], sq = a8[0] * bq8[0];
#pragma unroll
      for (int e = 1; e < 8; e++) { sk = fmaf(a8[e], bk8[e], sk); sq = fmaf(a8[e], bq8[e], sq); }
      sk = tree16(sk);
      sq = tree16(sq);
      if (c == 0 && jown < total) { sm.pk[j] = sk; sm.pq[j] = sq; }
    }
  }
  team_sync();                               // digit planes (and projections) are complete

  // (6) the state stream on the tensor cores
  {
    uint4 bf[2];
#pragma unroll
    for (int pp = 0; pp < 2; pp++) bf[pp] = *reinterpret_cast<const uint4 *>(sm.digits + g * D + 64 * pp + 16 * t);
#pragma unroll
    for (int mt = 0; mt < 2; mt++) {
      int c4[4] = {0, 0, 0, 0};
#pragma unroll
      for (int pp = 0; pp < 2; pp++) {
        mma_s8(c4, zlo[mt][pp].x, zhi[mt][pp].x, zlo[mt][pp].y, zhi[mt][pp].y, bf[pp].x, bf[pp].y);
        mma_s8(c4, zlo[mt][pp].z, zhi[mt][pp].z, zlo[mt][pp].w, zhi[mt][pp].w, bf[pp].z, bf[pp].w);
      }
      // c4[0], c4[1]: row g, planes 2t, 2t+1;  c4[2], c4[3]: row g+8.  Planes 4v..4v+3 are the digits of
      // vector v, so lanes t = 0, 1 carry the k sums and t = 2, 3 the q sums: even t the low digit pair.
      long long lo = static_cast<long long>(c4[0]) + (static_cast<long long>(c4[1]) << 8);
      long long hi = static_cast<long long>(c4[2]) + (static_cast<long long>(c4[3]) << 8);
      if (t & 1) { lo <<= 16; hi <<= 16; }
      lo += __shfl_xor_sync(FULL, lo, 1);
      hi += __shfl_xor_sync(FULL, hi, 1);
      if (!(t & 1)) {
        float *dst = (t & 2) ? sm.yq : sm.yk;
        const int j = 32 * warp + 16 * mt + g;
        dst[j] = __ll2float_rn(lo);
        dst[j + 8] = __ll2float_rn(hi);
      }
    }
  }
  team_sync();

  // (7) per value channel j = tid: scale the sums, add compensator and record terms, emit u and o
  {
    const int j = tid;
    float rk = s_j * (sm.yk[j] * back_k), rq = s_j * (sm.yq[j] * back_q);
    for (int h = 0; h < r; h++) {
      const float uc = sm.cu[h * D + j];
      rk = fmaf(uc, sm.pk[n + h], rk);
      rq = fmaf(uc, sm.pq[n + h], rq);
    }
    for (int jj = 0; jj < n; jj++) {
      const float uj = sm.bu[jj * D + j];
      rk = fmaf(uj, sm.pk[jj], rk);
      rq = fmaf(uj, sm.pq[jj], rq);
    }
    const float u = v_j - rk;
    const float o = fmaf(u, sm.pq[n + r], rq);
    p.o[bh * D + j] = o;
    p.buf_u[(bh * W + n) * (size_t)D + j] = u;
    p.buf_k[(bh * W + n) * (size_t)D + j] = kt_i;
    if (GATE == LQ_GATE_DIAG) p.buf_a[(bh * W + n) * (size_t)D + j] = a_i;
    else if (tid == 0) p.buf_a[bh * W + n] = a_i;
  }
}

template <int GATE>
__global__ void __launch_bounds__(128) decode_kernel(const Params p) {
  extern __shared__ float4 lq_smem4[];
  const DecodeSmem sm(reinterpret_cast<float *>(lq_smem4), p.W, p.r, GATE == LQ_GATE_DIAG);
  const size_t bh = blockIdx.x;
  const int b = static_cast<int>(bh / p.heads_v);
  const int n = p.win_pos[b] & 0xFFFF;       // bits 16.. are the arrival counter of this launch
  if (n >= p.W) return;                      // nothing can be appended: the sequence gets no token
  decode_head<GATE>(p, sm, bh, threadIdx.x, 1, n);
  __syncthreads();
  if (threadIdx.x == 0) arrive_and_set(p.win_pos, b, p.heads_v, n + 1);
}

}  // namespace lq
