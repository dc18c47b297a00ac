// Decode: one token for one (sequence, value head), done by ONE WARP.
//
// Eq. 10 (readout of the smoothed, compensated window representation) evaluated for x = alpha.k and
// x = alpha.q in one pass over the 8-bit codes:
//   S_{l-1}^T (alpha.x) = (B/127) Z^T (C Gamma_{1:l} x) + Uc (Kc^T Gamma_{1:l} x) + sum_j u_j (kt_j^T Gamma_{j+1:l} x)
// then u = v - S_{l-1}^T(alpha.k) (Eq. 3), o = S_{l-1}^T(alpha.q) + u (kt^T q), and the record is appended.
//
// Data movement: everything a head needs (16 KiB of codes, the two scale vectors, the compensators and the
// n buffered records) is brought into the warp's own shared-memory slot by TMA bulk copies that complete on
// an mbarrier; the warp loads the token's vectors meanwhile, waits once, and computes out of shared memory.
// A warp therefore keeps a whole head (about 27 KB at W = 16) in flight, and nothing in the kernel needs a
// CTA-wide barrier: warps are independent workers that walk over the heads with a grid stride.
//
// Arithmetic: the first term is a dense int8 contraction, Z^T [128 x 128] against the two vectors.  The
// vectors are put on a 30-bit block fixed-point grid and split into four signed base-256 digits each, which
// gives an int8 operand of 128 x 8; the tensor cores (mma.sync m16n8k32, s8 x s8 -> s32) produce exact
// integer sums, recombined in 64-bit integers and rounded to fp32 once, so the result does not depend on
// the order of accumulation.  The codes are stored value-channel major (Z^T, [d_v][d_k]): the contraction
// index is then contiguous, as the MMA operand layout needs.  The small dot products against records and
// compensators run on the fp32 pipes in the library's fixed summation order.
#pragma once
#include "lq_common.cuh"

namespace lq {

// Set when a bounded wait gave up (bit 0: a decode warp's wait for its bulk copies).  Never cleared by kernels.
__device__ int g_device_error = 0;

// ---- per-warp shared-memory slot ----
struct DecodeSlot {
  // byte offsets inside a slot; every region starts on a 16-byte boundary
  int zt, cs, bs, ck, cu, bk, bu, ba, digits, y, pk, pq, gs, mbar, bytes;
  __host__ __device__ DecodeSlot(int W, int r, bool diag) {
    int o = 0;
    zt = o; o += D * D;                 // codes, Z^T
    cs = o; o += 4 * D;                 // row_smooth
    bs = o; o += 4 * D;                 // col_scale
    ck = o; o += 2 * D * r;             // compensator keys, fp16
    cu = o; o += 2 * D * r;             // compensator values, fp16
    bk = o; o += 4 * D * W;             // buffered write keys
    bu = o; o += 4 * D * W;             // buffered corrections
    ba = o; o += diag ? 4 * D * W : 0;  // buffered diagonal decays, turned in place into Gamma_{j+1:l}
    digits = o; o += 8 * D;             // digit planes: plane 4v+d = digit d of vector v (0: k, 1: q)
    y = o; o += 2 * 4 * D;              // exact integer sums of the state stream, rounded to fp32: [2][128]
    pk = o; o += 4 * (MAX_W + MAX_R + 16);
    pq = o; o += 4 * (MAX_W + MAX_R + 16);   // projections; pq[n+r] holds kt^T q
    gs = o; o += 4 * MAX_W;             // scalar-gate decays Gamma_{j+1:l}
    mbar = o; o += 16;
    bytes = (o + 127) / 128 * 128;
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

// ---- mbarrier / TMA bulk copy (1-D) ----
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> shared bulk copy; addresses and size are multiples of 16 bytes
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// Bounded wait for phase `parity`; false if the limit ran out (the caller then reports and bails out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int spin = 0; spin < (1 << 20); spin++) {
    uint32_t done;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

__device__ __forceinline__ void widen8_bf16(const uint4 w, float (&x)[8]) {
  const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int e = 0; e < 4; e++) {
    x[2 * e] = __uint_as_float(ws[e] << 16);
    x[2 * e + 1] = __uint_as_float(ws[e] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void widen8_f16(const uint4 w, float (&x)[8]) {
  const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int e = 0; e < 4; e++) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&ws[e]));
    x[2 * e] = f.x;
    x[2 * e + 1] = f.y;
  }
}

// Persistent kernel of one-warp CTAs: warp `gw` of the grid takes heads gw, gw + nwarps, ...
template <int GATE>
__global__ void __launch_bounds__(32) decode_kernel(const Params p) {
  extern __shared__ __align__(128) unsigned char lq_smem_raw[];
  const int W = p.W, r = p.r;
  const DecodeSlot L(W, r, GATE == LQ_GATE_DIAG);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = lane & 15, half = lane >> 4, g = lane >> 2, t = lane & 3;
  unsigned char *slot = lq_smem_raw + (size_t)warp * L.bytes;
  const int8_t *zt = reinterpret_cast<const int8_t *>(slot + L.zt);
  const float *cs = reinterpret_cast<const float *>(slot + L.cs), *bs = reinterpret_cast<const float *>(slot + L.bs);
  const uint16_t *ckh = reinterpret_cast<const uint16_t *>(slot + L.ck), *cuh = reinterpret_cast<const uint16_t *>(slot + L.cu);
  const float *bk = reinterpret_cast<const float *>(slot + L.bk), *bu = reinterpret_cast<const float *>(slot + L.bu);
  float *ba = reinterpret_cast<float *>(slot + L.ba);
  int8_t *digits = reinterpret_cast<int8_t *>(slot + L.digits);
  float *y = reinterpret_cast<float *>(slot + L.y), *pk = reinterpret_cast<float *>(slot + L.pk);
  float *pq = reinterpret_cast<float *>(slot + L.pq), *gs = reinterpret_cast<float *>(slot + L.gs);
  const uint32_t bar = smem_addr(slot + L.mbar), slot_a = smem_addr(slot);

  if (lane == 0) mbar_init(bar, 1);
  __syncwarp();
  uint32_t parity = 0;

  const size_t nh = (size_t)p.batch * p.heads_v;
  const size_t nwarps = (size_t)gridDim.x * (blockDim.x >> 5);
  const int group = p.heads_v / p.heads_qk;

  for (size_t bh = (size_t)blockIdx.x * (blockDim.x >> 5) + warp; bh < nh; bh += nwarps) {
    const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);
    const int n = p.win_pos[b] & 0xFFFF;     // bits 16.. are the arrival counter of this launch
    if (n >= W) continue;                    // nothing can be appended: the sequence gets no token

    // (1) request the head: bulk copies into the slot, completion counted in bytes on the mbarrier
    if (lane == 0) {
      // the slot was last touched through ordinary loads and stores; order them before the async writes
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      const uint32_t rec = 4u * D * n;
      uint32_t total = D * D + 8u * D + 4u * D * r + 2u * rec + (GATE == LQ_GATE_DIAG ? rec : 0u);
      mbar_expect_tx(bar, total);
      bulk_g2s(slot_a + L.zt, p.codes + bh * (size_t)(D * D), D * D, bar);
      bulk_g2s(slot_a + L.cs, p.row_smooth + bh * D, 4 * D, bar);
      bulk_g2s(slot_a + L.bs, p.col_scale + bh * D, 4 * D, bar);
      if (r > 0) {
        bulk_g2s(slot_a + L.ck, p.comp_k + bh * (size_t)(r * D), 2 * D * r, bar);
        bulk_g2s(slot_a + L.cu, p.comp_u + bh * (size_t)(r * D), 2 * D * r, bar);
      }
      if (n > 0) {
        bulk_g2s(slot_a + L.bk, p.buf_k + bh * (size_t)(W * D), rec, bar);
        bulk_g2s(slot_a + L.bu, p.buf_u + bh * (size_t)(W * D), rec, bar);
        if (GATE == LQ_GATE_DIAG) bulk_g2s(slot_a + L.ba, p.buf_a + bh * (size_t)(W * D), rec, bar);
      }
    }

    // (2) the token, straight into registers.  Lane c (and its twin c+16) owns key channels 8c..8c+7;
    // lane l owns value channels 4l..4l+3.
    float k8[8], q8[8], kt8[8], a8[8], v4[4];
    {
      const size_t qk_off = ((size_t)b * p.heads_qk + hv / group) * D;
      widen8_bf16(*reinterpret_cast<const uint4 *>(p.k + qk_off + 8 * c), k8);
      widen8_bf16(*reinterpret_cast<const uint4 *>(p.q + qk_off + 8 * c), q8);
      const uint2 vw = *reinterpret_cast<const uint2 *>(p.v + bh * D + 4 * lane);
      v4[0] = __uint_as_float(vw.x << 16); v4[1] = __uint_as_float(vw.x & 0xFFFF0000u);
      v4[2] = __uint_as_float(vw.y << 16); v4[3] = __uint_as_float(vw.y & 0xFFFF0000u);
      const float beta = bf16_bits(p.beta[bh]);
      if (GATE == LQ_GATE_DIAG) {
        widen8_bf16(*reinterpret_cast<const uint4 *>(p.alpha + bh * D + 8 * c), a8);
      } else {
        const float a = bf16_bits(p.alpha[bh]);
#pragma unroll
        for (int e = 0; e < 8; e++) a8[e] = a;
      }
#pragma unroll
      for (int e = 0; e < 8; e++) kt8[e] = beta * k8[e];
    }
    float ba_lo = 1.0f, ba_hi = 1.0f;        // scalar gate: decay of record `lane` and of record `lane + 32`
    if (GATE == LQ_GATE_SCALAR) {
      if (lane < n) ba_lo = p.buf_a[bh * (size_t)W + lane];
      if (lane + 32 < n) ba_hi = p.buf_a[bh * (size_t)W + lane + 32];
    }

    // (3) wait for the slot (bounded: a copy that never lands must not hang the GPU)
    if (!mbar_wait(bar, parity)) {
      if (lane == 0) atomicOr(&g_device_error, 1);
      mbar_wait(bar, parity);                // one more bounded wait for the copies in flight, then give up
      return;
    }
    parity ^= 1u;

    // (4) cumulative decays from the newest record back (Appendix B.2).  After the loop g8 = Gamma_{1:l}.
    float g8[8];
#pragma unroll
    for (int e = 0; e < 8; e++) g8[e] = a8[e];
    if (GATE == LQ_GATE_DIAG) {
      for (int j = n - 1; j >= 0; j--) {
        float aj[8];
        load8(ba + j * D + 8 * c, aj);
        __syncwarp();                        // both twins have read the decay before one of them replaces it
        if (half == 0) store8(ba + j * D + 8 * c, g8);   // Gamma_{j+1:l} in place of the record's decay
#pragma unroll
        for (int e = 0; e < 8; e++) g8[e] = g8[e] * aj[e];
      }
    } else {
      float gsc = a8[0];
      for (int j = n - 1; j >= 0; j--) {     // every lane runs the same scalar chain
        if (lane == (j & 31)) gs[j] = gsc;
        gsc = gsc * __shfl_sync(FULL, j < 32 ? ba_lo : ba_hi, j & 31);
      }
#pragma unroll
      for (int e = 0; e < 8; e++) g8[e] = gsc;
    }
    float gk8[8], gq8[8];
#pragma unroll
    for (int e = 0; e < 8; e++) { gk8[e] = g8[e] * k8[e]; gq8[e] = g8[e] * q8[e]; }

    // (4b) C Gamma k (lanes 0..15) and C Gamma q (lanes 16..31) on their fixed-point grids, as digit planes
    float back_own;
    {
      float c8[8], x8[8];
      load8(cs + 8 * c, c8);
      float m = 0.0f;
#pragma unroll
      for (int e = 0; e < 8; e++) {
        x8[e] = c8[e] * (half ? gq8[e] : gk8[e]);
        m = fmaxf(m, fabsf(x8[e]));
      }
#pragma unroll
      for (int s = 1; s <= 8; s <<= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, s));
      float scale;
      fixed_point_scales(m, scale, back_own);
      uint32_t lo[4] = {0u, 0u, 0u, 0u}, hi[4] = {0u, 0u, 0u, 0u};      // [digit]: bytes of elements 0..3 / 4..7
#pragma unroll
      for (int e = 0; e < 8; e++) {
        int X = __float2int_rn(x8[e] * scale);
#pragma unroll
        for (int d = 0; d < 4; d++) {       // X = d0 + 256 d1 + 65536 d2 + 2^24 d3, digits in [-128, 127]
          const int dig = (X << 24) >> 24;
          const uint32_t byte = static_cast<uint32_t>(dig) & 0xFFu;
          if (e < 4) lo[d] |= byte << (8 * e); else hi[d] |= byte << (8 * (e - 4));
          X = (X - dig) >> 8;
        }
      }
#pragma unroll
      for (int d = 0; d < 4; d++)
        *reinterpret_cast<uint2 *>(digits + (4 * half + d) * D + 8 * c) = make_uint2(lo[d], hi[d]);
    }
    const float back_other = __shfl_xor_sync(FULL, back_own, 16);
    const float back_k = half ? back_other : back_own, back_q = half ? back_own : back_other;
    __syncwarp();                            // in-place decays, gs and digit planes are visible to the warp

    // (5) projections: the two halves of the warp take one dot-product pair each per trip (lane c owns block
    // c of eight terms).  Both halves make the same number of trips: the shuffles name all 32 lanes.
    {
      const int total = n + r + 1;
      for (int jb = 0; jb < total; jb += 2) {
        const int jown = jb + half;
        const int j = jown < total ? jown : total - 1;
        float x8[8], yk8[8], yq8[8];
        if (j < n) {
          load8(bk + j * D + 8 * c, x8);
          if (GATE == LQ_GATE_DIAG) {
            float gj8[8];
            load8(ba + j * D + 8 * c, gj8);
#pragma unroll
            for (int e = 0; e < 8; e++) { yk8[e] = gj8[e] * k8[e]; yq8[e] = gj8[e] * q8[e]; }
          } else {
            const float gj = gs[j];
#pragma unroll
            for (int e = 0; e < 8; e++) { yk8[e] = gj * k8[e]; yq8[e] = gj * q8[e]; }
          }
        } else if (j < n + r) {
          widen8_f16(*reinterpret_cast<const uint4 *>(ckh + (j - n) * D + 8 * c), x8);
#pragma unroll
          for (int e = 0; e < 8; e++) { yk8[e] = gk8[e]; yq8[e] = gq8[e]; }
        } else {                             // kt^T q, kept in the pq slot; the pk slot is unused
#pragma unroll
          for (int e = 0; e < 8; e++) { x8[e] = kt8[e]; yk8[e] = q8[e]; yq8[e] = q8[e]; }
        }
        float sk = x8[0] * yk8[0], sq = x8[0] * yq8[0];
#pragma unroll
        for (int e = 1; e < 8; e++) { sk = fmaf(x8[e], yk8[e], sk); sq = fmaf(x8[e], yq8[e], sq); }
        sk = tree16(sk);
        sq = tree16(sq);
        if (c == 0 && jown < total) { pk[j] = sk; pq[j] = sq; }
      }
    }

    // (6) the state stream on the tensor cores: eight 16-row tiles of Z^T, K = 128 as four k-blocks.
    // A thread's 16 bytes of a row hold key channels 64p+16t..64p+16t+15 and serve two k-blocks; the digit
    // planes are read with the same permutation of the key index.
    {
      uint4 bf[2];
#pragma unroll
      for (int pp = 0; pp < 2; pp++) bf[pp] = *reinterpret_cast<const uint4 *>(digits + g * D + 64 * pp + 16 * t);
#pragma unroll 2
      for (int mt = 0; mt < 8; mt++) {
        int c4[4] = {0, 0, 0, 0};
        const int j = 16 * mt + g;
#pragma unroll
        for (int pp = 0; pp < 2; pp++) {
          const uint4 zlo = *reinterpret_cast<const uint4 *>(zt + j * D + 64 * pp + 16 * t);
          const uint4 zhi = *reinterpret_cast<const uint4 *>(zt + (j + 8) * D + 64 * pp + 16 * t);
          mma_s8(c4, zlo.x, zhi.x, zlo.y, zhi.y, bf[pp].x, bf[pp].y);
          mma_s8(c4, zlo.z, zhi.z, zlo.w, zhi.w, bf[pp].z, bf[pp].w);
        }
        // c4[0], c4[1]: row g, planes 2t, 2t+1;  c4[2], c4[3]: row g+8.  Planes 4v..4v+3 are the digits of
        // vector v: lanes t = 0, 1 carry the k sums and t = 2, 3 the q sums, even t the low digit pair.
        long long lo = static_cast<long long>(c4[0]) + (static_cast<long long>(c4[1]) << 8);
        long long hi = static_cast<long long>(c4[2]) + (static_cast<long long>(c4[3]) << 8);
        if (t & 1) { lo <<= 16; hi <<= 16; }
        lo += __shfl_xor_sync(FULL, lo, 1);
        hi += __shfl_xor_sync(FULL, hi, 1);
        if (!(t & 1)) {
          float *dst = y + (t >> 1) * D;
          dst[j] = __ll2float_rn(lo);
          dst[j + 8] = __ll2float_rn(hi);
        }
      }
    }
    __syncwarp();

    // (7) per value channel (lane l: channels 4l..4l+3): scale the sums, add compensator and record terms
    {
      const float4 yk4 = *reinterpret_cast<const float4 *>(y + 4 * lane);
      const float4 yq4 = *reinterpret_cast<const float4 *>(y + D + 4 * lane);
      const float4 b4 = *reinterpret_cast<const float4 *>(bs + 4 * lane);
      const float s4[4] = {b4.x / 127.0f, b4.y / 127.0f, b4.z / 127.0f, b4.w / 127.0f};
      float rk[4] = {s4[0] * (yk4.x * back_k), s4[1] * (yk4.y * back_k), s4[2] * (yk4.z * back_k), s4[3] * (yk4.w * back_k)};
      float rq[4] = {s4[0] * (yq4.x * back_q), s4[1] * (yq4.y * back_q), s4[2] * (yq4.z * back_q), s4[3] * (yq4.w * back_q)};
      for (int h = 0; h < r; h++) {
        const uint2 w = *reinterpret_cast<const uint2 *>(cuh + h * D + 4 * lane);
        const float2 f01 = __half22float2(*reinterpret_cast<const __half2 *>(&w.x));
        const float2 f23 = __half22float2(*reinterpret_cast<const __half2 *>(&w.y));
        const float uc[4] = {f01.x, f01.y, f23.x, f23.y};
        const float pkh = pk[n + h], pqh = pq[n + h];
#pragma unroll
        for (int e = 0; e < 4; e++) { rk[e] = fmaf(uc[e], pkh, rk[e]); rq[e] = fmaf(uc[e], pqh, rq[e]); }
      }
      for (int jj = 0; jj < n; jj++) {
        const float4 u4 = *reinterpret_cast<const float4 *>(bu + jj * D + 4 * lane);
        const float uj[4] = {u4.x, u4.y, u4.z, u4.w};
        const float pkj = pk[jj], pqj = pq[jj];
#pragma unroll
        for (int e = 0; e < 4; e++) { rk[e] = fmaf(uj[e], pkj, rk[e]); rq[e] = fmaf(uj[e], pqj, rq[e]); }
      }
      const float ktq = pq[n + r];
      float u[4], o[4];
#pragma unroll
      for (int e = 0; e < 4; e++) { u[e] = v4[e] - rk[e]; o[e] = fmaf(u[e], ktq, rq[e]); }
      *reinterpret_cast<float4 *>(p.o + bh * D + 4 * lane) = make_float4(o[0], o[1], o[2], o[3]);
      *reinterpret_cast<float4 *>(p.buf_u + (bh * W + n) * (size_t)D + 4 * lane) = make_float4(u[0], u[1], u[2], u[3]);
      if (half == 0) {
        store8(p.buf_k + (bh * W + n) * (size_t)D + 8 * c, kt8);
        if (GATE == LQ_GATE_DIAG) store8(p.buf_a + (bh * W + n) * (size_t)D + 8 * c, a8);
        else if (lane == 0) p.buf_a[bh * W + n] = a8[0];
      }
    }
    __syncwarp();
    if (lane == 0) arrive_and_set(p.win_pos, b, p.heads_v, n + 1);
  }
}

}  // namespace lq
