// Decode kernel: one token for one (sequence, value head) per CTA of 128 threads.
//
// Eq. 10 (readout of the smoothed, compensated window representation) evaluated for x = alpha.k and
// x = alpha.q in one pass over the 8-bit codes:
//   S_{l-1}^T (alpha.x) = (B/127) Z^T (C Gamma_{1:l} x) + Uc (Kc^T Gamma_{1:l} x) + sum_j u_j (kt_j^T Gamma_{j+1:l} x)
// then u = v - S_{l-1}^T(alpha.k) (Eq. 3), o = S_{l-1}^T(alpha.q) + u (kt^T q), and the record is appended.
//
// The 16 KiB of codes are the bulk of the traffic.  Thread (ty, tx) = (tid >> 3, tid & 7) owns rows
// 8ty..8ty+7 and columns 16tx..16tx+15: eight independent 16-byte loads issued at kernel entry, consumed
// after the (much smaller) record walk, so that a CTA has its whole state in flight at once.
#pragma once
#include "lq_common.cuh"

namespace lq {

struct DecodeSmem {
  float *bk, *bu, *ba;      // staged records: [W][128], [W][128], [W][128] (diag) or [MAX_W] (scalar)
  float *ck, *cu;           // compensators widened to fp32: [r][128] each
  float *kf, *qf, *kt;      // token vectors
  float *gk, *gq;           // Gamma_{1:l} k, Gamma_{1:l} q
  float *xk, *xq;           // C Gamma_{1:l} k, C Gamma_{1:l} q
  float *part;              // [4 warps][2][128] column partial sums
  float *pk, *pq;           // [MAX_W + MAX_R + 1] projections; the last used slot holds kt^T q
  float *gs;                // [MAX_W] scalar-gate decays Gamma_{j+1:l}
  __device__ __forceinline__ DecodeSmem(float *base, int W, int r, bool diag) {
    bk = base; bu = bk + W * D; ba = bu + W * D; ck = ba + (diag ? W * D : MAX_W); cu = ck + r * D;
    kf = cu + r * D; qf = kf + D; kt = qf + D; gk = kt + D; gq = gk + D; xk = gq + D; xq = xk + D;
    part = xq + D; pk = part + 4 * 2 * D; pq = pk + (MAX_W + MAX_R + 16); gs = pq + (MAX_W + MAX_R + 16);
  }
  static size_t bytes(int W, int r, bool diag) {
    return sizeof(float) * (size_t)(2 * W * D + (diag ? W * D : MAX_W) + 2 * r * D + 7 * D + 8 * D +
                                    2 * (MAX_W + MAX_R + 16) + MAX_W);
  }
};

template <int GATE>
__global__ void __launch_bounds__(128) decode_kernel(const Params p) {
  extern __shared__ float4 lq_smem4[];
  const int W = p.W, r = p.r;
  const DecodeSmem sm(reinterpret_cast<float *>(lq_smem4), W, r, GATE == LQ_GATE_DIAG);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, ty = tid >> 3, tx = tid & 7;
  const size_t bh = blockIdx.x;
  const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);

  // (1) the codes: everything this thread will need of Z
  uint4 z[8];
  {
    const int8_t *Z = p.codes + bh * (size_t)(D * D);
#pragma unroll
    for (int m = 0; m < 8; m++) z[m] = *reinterpret_cast<const uint4 *>(Z + (8 * ty + m) * D + 16 * tx);
  }
  const int n = p.win_pos[b] & 0xFFFF;       // bits 16.. are the arrival counter of this launch
  if (n >= W) return;                        // nothing can be appended: the sequence is left untouched

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
  __syncthreads();

  // (4) cumulative decays from the newest record back (Appendix B.2).  After the loop g = Gamma_{1:l}.
  float g = a_i;
  if (GATE == LQ_GATE_DIAG) {
    for (int j = n - 1; j >= 0; j--) {
      const float aj = sm.ba[j * D + tid];
      sm.ba[j * D + tid] = g;              // Gamma_{j+1:l} for channel i, in place of the record's decay
      g = g * aj;
    }
  } else {
    for (int j = n - 1; j >= 0; j--) {     // every thread runs the same scalar chain
      if (tid == 0) sm.gs[j] = g;
      g = g * sm.ba[j];
    }
  }
  {
    const float gk = g * k_i, gq = g * q_i;
    sm.gk[tid] = gk; sm.gq[tid] = gq;
    sm.xk[tid] = c_i * gk; sm.xq[tid] = c_i * gq;
  }
  __syncthreads();

  // (5) projections: one dot product pair per group of sixteen lanes (lane c owns block c of eight terms)
  {
    // The trip count is the same for both halves of a warp (the shuffles of tree16 name all 32 lanes):
    // a half without a dot product of its own recomputes the last one and does not store it.
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

  // (6) the state stream: column sums of Z against xk and xq, block of eight rows per thread
  float accK[16], accQ[16];
  {
    float xk8[8], xq8[8];
    load8(sm.xk + 8 * ty, xk8);
    load8(sm.xq + 8 * ty, xq8);
#pragma unroll
    for (int m = 0; m < 8; m++) {
      const uint32_t wds[4] = {z[m].x, z[m].y, z[m].z, z[m].w};
#pragma unroll
      for (int cc = 0; cc < 16; cc++) {
        const float zf = static_cast<float>(static_cast<int8_t>((wds[cc >> 2] >> (8 * (cc & 3))) & 0xFF));
        if (m == 0) { accK[cc] = zf * xk8[0]; accQ[cc] = zf * xq8[0]; }
        else { accK[cc] = fmaf(zf, xk8[m], accK[cc]); accQ[cc] = fmaf(zf, xq8[m], accQ[cc]); }
      }
    }
  }
  // tree over the sixteen row blocks: ty^1 is lane^8, ty^2 is lane^16, then warps through shared memory.
  // Halving exchanges: lanes with bit 3 clear end up with the k sums, the others with the q sums.
  {
    const bool up8 = lane & 8, up16 = lane & 16;
    float h16[16], h8[8];
#pragma unroll
    for (int e = 0; e < 16; e++) {
      const float keep = up8 ? accQ[e] : accK[e], send = up8 ? accK[e] : accQ[e];
      h16[e] = keep + __shfl_xor_sync(FULL, send, 8);
    }
#pragma unroll
    for (int e = 0; e < 8; e++) {
      const float keep = up16 ? h16[e + 8] : h16[e], send = up16 ? h16[e] : h16[e + 8];
      h8[e] = keep + __shfl_xor_sync(FULL, send, 16);
    }
    store8(sm.part + (warp * 2 + (up8 ? 1 : 0)) * D + 16 * tx + (up16 ? 8 : 0), h8);
  }
  __syncthreads();

  // (7) per value channel j = tid: finish the sums, add compensator and record terms, emit u and o
  {
    const int j = tid;
    const float yk = (sm.part[(0 * 2 + 0) * D + j] + sm.part[(1 * 2 + 0) * D + j]) +
                     (sm.part[(2 * 2 + 0) * D + j] + sm.part[(3 * 2 + 0) * D + j]);
    const float yq = (sm.part[(0 * 2 + 1) * D + j] + sm.part[(1 * 2 + 1) * D + j]) +
                     (sm.part[(2 * 2 + 1) * D + j] + sm.part[(3 * 2 + 1) * D + j]);
    float rk = s_j * yk, rq = s_j * yq;
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
  __syncthreads();
  if (tid == 0) arrive_and_set(p.win_pos, b, p.heads_v, n + 1);
}

}  // namespace lq
