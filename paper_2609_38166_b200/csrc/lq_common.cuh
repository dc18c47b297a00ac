// Device helpers shared by the sm_100a kernels of the per-window 8-bit decode step.
//
// Everything is compiled with -fmad=false: a product is fused with an addition only where fmaf() is
// written, so that every value is reproducible bit for bit.  Sums over a channel index follow one
// fixed order: the terms are taken in blocks of eight; inside a block the even- and the odd-numbered
// terms form two chains, each accumulated left to right (first product rounded, the rest folded in with
// fmaf), and the two chains are added; block results are added as a balanced binary tree over the block
// index.  The thread mappings below are chosen so that this order is the natural one: a thread owns one
// block of eight (where registers allow, as four float2 pairs, so that one packed fused multiply-add,
// FFMA2 on sm_100, advances both chains); neighbouring lanes own neighbouring blocks, and butterfly
// exchanges with lane masks 1, 2, 4, ... walk up the tree.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lq.h"

namespace lq {

constexpr int D = 128;       // d_k = d_v of the supported shape
constexpr int MAX_W = 64;
constexpr int MAX_R = 16;
constexpr unsigned FULL = 0xffffffffu;

// Byte offsets inside a head block and float offsets inside a record row (d_k = d_v = 128).
constexpr int HB_CODES = 0;
constexpr int HB_COL_SCALE = D * D;
constexpr int HB_ROW_SMOOTH = HB_COL_SCALE + 4 * D;
constexpr int HB_COMP_K = HB_ROW_SMOOTH + 4 * D;
__host__ __device__ constexpr int hb_comp_u(int r) { return HB_COMP_K + 2 * D * r; }
__host__ __device__ constexpr int head_bytes(int r) { return HB_COMP_K + 4 * D * r; }
__host__ __device__ constexpr int record_floats(bool diag) { return diag ? 3 * D : 2 * D; }
constexpr int REC_KT = 0, REC_U = D, REC_A = 2 * D;

// Launch-time description of one call, passed to the kernels by value.
struct Params {
  int batch, heads_v, heads_qk, W, r, n_iter, smooth, delta, rec16, force;
  uint8_t *heads;    // [B*Hv] head blocks of head_bytes(r)
  void *records;     // [B*Hv][W] record rows of record_floats(gate) elements, fp32 or (rec16) fp16
  float *decays;     // scalar gate: [B*Hv][W]
  int32_t *win_pos;
  int32_t *work;     // lq_state.work (scratch words, zero between calls), or null
  const uint16_t *q, *k, *v, *beta, *alpha;
  float *o;
  float *S;          // dense fp32 states (quantize / dequantize / fp32 baseline)
  uint16_t *S16;     // dense bf16 states (bf16 baseline)
#ifdef LQ_TIMING
  int gen;           // development aid: which of the four generations of time stamps this launch writes
#endif

  __device__ __forceinline__ uint8_t *head(size_t bh) const { return heads + bh * (size_t)head_bytes(r); }
  __device__ __forceinline__ int8_t *codes(size_t bh) const { return reinterpret_cast<int8_t *>(head(bh) + HB_CODES); }
  __device__ __forceinline__ float *col_scale(size_t bh) const { return reinterpret_cast<float *>(head(bh) + HB_COL_SCALE); }
  __device__ __forceinline__ float *row_smooth(size_t bh) const { return reinterpret_cast<float *>(head(bh) + HB_ROW_SMOOTH); }
  __device__ __forceinline__ uint16_t *comp_k(size_t bh) const { return reinterpret_cast<uint16_t *>(head(bh) + HB_COMP_K); }
  __device__ __forceinline__ uint16_t *comp_u(size_t bh) const { return reinterpret_cast<uint16_t *>(head(bh) + hb_comp_u(r)); }
  // row of record j of head bh; `diag` selects the row length, T the element type (float, or __half with rec16)
  template <typename T>
  __device__ __forceinline__ T *record(size_t bh, int j, bool diag) const {
    return static_cast<T *>(records) + (bh * W + j) * (size_t)record_floats(diag);
  }
};

__device__ __forceinline__ float bf16_bits(uint16_t h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }
__device__ __forceinline__ float f16_bits(uint16_t h) { return __half2float(__ushort_as_half(h)); }
// binary32 -> binary16 bits, nearest even, clamped to the finite range first
__device__ __forceinline__ uint16_t to_f16_bits_sat(float x) {
  x = fminf(fmaxf(x, -65504.0f), 65504.0f);
  return __half_as_ushort(__float2half_rn(x));
}
// binary32 -> bfloat16 bits, nearest even (finite inputs)
__device__ __forceinline__ uint16_t to_bf16_bits(float x) {
  uint32_t u = __float_as_uint(x);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return static_cast<uint16_t>(u >> 16);
}

// ---- asynchronous global -> shared copies (16 bytes each) ----
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
  unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
// L2 eviction priorities: lines that will not be read again soon / lines another kernel reads next
__device__ __forceinline__ uint64_t l2_stream_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ uint64_t l2_keep_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ void cp_async4(void *smem, const void *gmem) {
  unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }
// all but the most recently committed group have landed
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;\n" ::: "memory"); }

// ---- sum of sixteen block results held by sixteen neighbouring lanes (tree levels 1, 2, 4, 8) ----
__device__ __forceinline__ float tree16(float x) {
  x = x + __shfl_xor_sync(FULL, x, 1);
  x = x + __shfl_xor_sync(FULL, x, 2);
  x = x + __shfl_xor_sync(FULL, x, 4);
  x = x + __shfl_xor_sync(FULL, x, 8);
  return x;
}

__device__ __forceinline__ float2 pair(float x) { return make_float2(x, x); }

// Block result of eight products a[e]*b[e] given as four pairs: the .x components are the even-numbered
// terms, the .y components the odd-numbered ones; each chain runs left to right, then the two are added.
__device__ __forceinline__ float block8(const float2 (&a)[4], const float2 (&b)[4]) {
  float2 acc = __fmul2_rn(a[0], b[0]);
#pragma unroll
  for (int c = 1; c < 4; c++) acc = __ffma2_rn(a[c], b[c], acc);
  return acc.x + acc.y;
}

__device__ __forceinline__ void load8p(const float *src, float2 (&x)[4]) {
  const float4 lo = *reinterpret_cast<const float4 *>(src), hi = *reinterpret_cast<const float4 *>(src + 4);
  x[0] = make_float2(lo.x, lo.y); x[1] = make_float2(lo.z, lo.w);
  x[2] = make_float2(hi.x, hi.y); x[3] = make_float2(hi.z, hi.w);
}
__device__ __forceinline__ void store8p(float *dst, const float2 (&x)[4]) {
  *reinterpret_cast<float4 *>(dst) = make_float4(x[0].x, x[0].y, x[1].x, x[1].y);
  *reinterpret_cast<float4 *>(dst + 4) = make_float4(x[2].x, x[2].y, x[3].x, x[3].y);
}

// Dot product of two 128-vectors in shared memory, computed by sixteen neighbouring lanes
// (lane c = lane & 15 owns block c); every one of the sixteen lanes returns the sum.
__device__ __forceinline__ float dot128_shared(const float *a, const float *b, int c) {
  float2 a2[4], b2[4];
  load8p(a + 8 * c, a2);
  load8p(b + 8 * c, b2);
  return tree16(block8(a2, b2));
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may become resident
// before the kernel ahead of it has finished; this is where it waits for that kernel's completion and writes
// (a no-op for an ordinary launch).  Right after it the kernel allows its own dependents to be scheduled.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Phase timing (development aid, compiled in with -DLQ_TIMING only): clock cycles per phase of the decode
// warps, summed over all heads by lane 0 of each warp (slots 0..15: stream warp, 16..31: dot warp; 32..: thread 0 of the boundary kernel's CTAs).
#ifdef LQ_TIMING
__device__ unsigned long long g_phase_cycles[64];
// cycles are summed in registers and flushed once per warp at the end of the kernel, so that the probe
// itself puts no traffic on the memory system while the kernel runs
// (-DLQ_STAMPS_ONLY: the per-CTA time stamps below without the per-phase counters, which cost ≈ 10 % of the time)
#ifdef LQ_STAMPS_ONLY
#define LQ_TICK(slot) do { } while (0)
#else
#define LQ_TICK(slot)                                     \
  do {                                                    \
    const long long now_ = clock64();                     \
    acc_[slot] += static_cast<unsigned>(now_ - tick_);    \
    tick_ = now_;                                         \
  } while (0)
#endif
// the boundary kernel's variant: thread 0 of the CTA keeps its sums in shared memory
__shared__ unsigned lq_bacc[16];
__shared__ long long lq_btick;
#ifdef LQ_STAMPS_ONLY
#define LQ_BTICK(slot) do { } while (0)
#else
#define LQ_BTICK(slot)                                          \
  do {                                                          \
    if (threadIdx.x == 0) {                                     \
      const long long now_ = clock64();                         \
      lq_bacc[slot] += static_cast<unsigned>(now_ - lq_btick);  \
      lq_btick = now_;                                          \
    }                                                           \
  } while (0)
#endif
// time stamps (ns, the GPU's global timer) of thread 0 of every CTA: [generation][kernel][stamp][CTA]
__device__ unsigned long long g_timeline[4][2][6][1024];
#define LQ_STAMP(kernel, slot)                                                                   \
  do {                                                                                           \
    if (threadIdx.x == 0 && blockIdx.x < 1024) {                                                 \
      unsigned long long t_;                                                                     \
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                      \
      g_timeline[p.gen & 3][kernel][slot][blockIdx.x] = t_;                                      \
    }                                                                                            \
  } while (0)
#else
#define LQ_TICK(slot) do { } while (0)
#define LQ_BTICK(slot) do { } while (0)
#define LQ_STAMP(kernel, slot) do { } while (0)
#endif

// =====================================================================================
// 8x8 register tiles: a CTA of 256 threads holds one 128x128 state, thread (ty, tx) owning rows
// 8ty..8ty+7 and columns 8tx..8tx+7, with tx = lane & 15 and ty = 2*warp + (lane >> 4).
// =====================================================================================
struct Tile {
  int tid, lane, warp, tx, ty;
  __device__ __forceinline__ Tile() {
    tid = threadIdx.x; lane = tid & 31; warp = tid >> 5; tx = lane & 15; ty = tid >> 4;
  }
};

__device__ __forceinline__ void load8(const float *src, float (&x)[8]) {
  const float4 lo = *reinterpret_cast<const float4 *>(src), hi = *reinterpret_cast<const float4 *>(src + 4);
  x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w; x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
}
__device__ __forceinline__ void store8(float *dst, const float (&x)[8]) {
  *reinterpret_cast<float4 *>(dst) = make_float4(x[0], x[1], x[2], x[3]);
  *reinterpret_cast<float4 *>(dst + 4) = make_float4(x[4], x[5], x[6], x[7]);
}

// ---- record rows kept in fp16: the same accessors on __half rows (widening is exact; narrowing saturates to
// the finite range and rounds to nearest even, like the compensators) ----
__device__ __forceinline__ void load8p(const __half *src, float2 (&x)[4]) {
  const uint4 raw = *reinterpret_cast<const uint4 *>(src);
  const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
  for (int i = 0; i < 4; i++) x[i] = __half22float2(h[i]);
}
__device__ __forceinline__ void load8(const __half *src, float (&x)[8]) {
  float2 v[4];
  load8p(src, v);
#pragma unroll
  for (int i = 0; i < 4; i++) { x[2 * i] = v[i].x; x[2 * i + 1] = v[i].y; }
}
__device__ __forceinline__ float4 load4(const float *src) { return *reinterpret_cast<const float4 *>(src); }
__device__ __forceinline__ float4 load4(const __half *src) {
  const uint2 raw = *reinterpret_cast<const uint2 *>(src);
  const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&raw.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&raw.y));
  return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ uint32_t pack2_f16_sat(float a, float b) {
  return (uint32_t)to_f16_bits_sat(a) | ((uint32_t)to_f16_bits_sat(b) << 16);
}
__device__ __forceinline__ void store8p(__half *dst, const float2 (&x)[4]) {
  *reinterpret_cast<uint4 *>(dst) = make_uint4(pack2_f16_sat(x[0].x, x[0].y), pack2_f16_sat(x[1].x, x[1].y),
                                               pack2_f16_sat(x[2].x, x[2].y), pack2_f16_sat(x[3].x, x[3].y));
}
__device__ __forceinline__ void store8(__half *dst, const float (&x)[8]) {
  *reinterpret_cast<uint4 *>(dst) = make_uint4(pack2_f16_sat(x[0], x[1]), pack2_f16_sat(x[2], x[3]),
                                               pack2_f16_sat(x[4], x[5]), pack2_f16_sat(x[6], x[7]));
}
__device__ __forceinline__ void store4(float *dst, float a, float b, float c, float d) {
  *reinterpret_cast<float4 *>(dst) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__half *dst, float a, float b, float c, float d) {
  *reinterpret_cast<uint2 *>(dst) = make_uint2(pack2_f16_sat(a, b), pack2_f16_sat(c, d));
}

// Row sums.  In: p[a] = this thread's block result for row 8ty+a (block index tx).
// Out: the full sum of row 8ty+sel, the same value in lanes tx and tx^8; sel depends on tx & 7 only.
// Halving exchanges: after the step with mask m a lane keeps the rows whose partner-combined sums it owns.
__device__ __forceinline__ float row_tree(const float (&p)[8], int lane, int &sel) {
  float q4[4], q2[2], q1;
  const bool u0 = lane & 1, u1 = lane & 2, u2 = lane & 4;
#pragma unroll
  for (int e = 0; e < 4; e++) {
    const float keep = u0 ? p[e + 4] : p[e], send = u0 ? p[e] : p[e + 4];
    q4[e] = keep + __shfl_xor_sync(FULL, send, 1);
  }
#pragma unroll
  for (int e = 0; e < 2; e++) {
    const float keep = u1 ? q4[e + 2] : q4[e], send = u1 ? q4[e] : q4[e + 2];
    q2[e] = keep + __shfl_xor_sync(FULL, send, 2);
  }
  {
    const float keep = u2 ? q2[1] : q2[0], send = u2 ? q2[0] : q2[1];
    q1 = keep + __shfl_xor_sync(FULL, send, 4);
  }
  q1 = q1 + __shfl_xor_sync(FULL, q1, 8);
  sel = (u0 ? 4 : 0) + (u1 ? 2 : 0) + (u2 ? 1 : 0);
  return q1;
}

// Column sums.  In: p[b] = this thread's block result for column 8tx+b (block index ty).
// part: 8*128 floats and out: 128 floats of shared memory.  Returns w[b] = full sum of column 8tx+b in
// every thread.  Tree levels: ty^1 inside the warp (lane^16), then warps (0,1)(2,3)(4,5)(6,7), pairs of
// pairs, halves.  Contains two __syncthreads(); `part` and `out` may be rewritten after the CTA's next barrier.
__device__ __forceinline__ void col_tree(const float (&p)[8], float *part, float *out, const Tile &t, float (&w)[8]) {
  const bool up = t.lane & 16;
  {
    float r[4];
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float keep = up ? p[e + 4] : p[e], send = up ? p[e] : p[e + 4];
      r[e] = keep + __shfl_xor_sync(FULL, send, 16);      // rows 16w..16w+7 with rows 16w+8..16w+15
    }
    *reinterpret_cast<float4 *>(part + t.warp * D + 8 * t.tx + (up ? 4 : 0)) = make_float4(r[0], r[1], r[2], r[3]);
  }
  __syncthreads();
  if (t.tid < D) {
    const float *c = part + t.tid;
    out[t.tid] = ((c[0] + c[D]) + (c[2 * D] + c[3 * D])) + ((c[4 * D] + c[5 * D]) + (c[6 * D] + c[7 * D]));
  }
  __syncthreads();
  load8(out + 8 * t.tx, w);
}

// p[b] = block result over this thread's eight rows of  sum_a M[a][b] * x[a]: rows 0,2,4,6 and rows
// 1,3,5,7 are the two chains of the block.  (Scalar operations: a packed one would need the per-row
// multiplier duplicated into a register pair, and the 64-register tile leaves no room for that.)
__device__ __forceinline__ void col_blocks(const float (&M)[8][8], const float (&x)[8], float (&p)[8]) {
#pragma unroll
  for (int b = 0; b < 8; b++) {
    float even = M[0][b] * x[0], odd = M[1][b] * x[1];
#pragma unroll
    for (int a = 2; a < 8; a += 2) {
      even = fmaf(M[a][b], x[a], even);
      odd = fmaf(M[a + 1][b], x[a + 1], odd);
    }
    p[b] = even + odd;
  }
}
// p[a] = block result over this thread's eight columns of  sum_b M[a][b] * x[b]
__device__ __forceinline__ void row_blocks(const float (&M)[8][8], const float (&x)[8], float (&p)[8]) {
#pragma unroll
  for (int a = 0; a < 8; a++) {
    float even = M[a][0] * x[0], odd = M[a][1] * x[1];
#pragma unroll
    for (int b = 2; b < 8; b += 2) {
      even = fmaf(M[a][b], x[b], even);
      odd = fmaf(M[a][b + 1], x[b + 1], odd);
    }
    p[a] = even + odd;
  }
}

// Last-arrival bookkeeping on win_pos[b]: bits 16.. count the heads of sequence b that are done with
// the value in bits 0..15.  The head that arrives last (all heads_v have read the old value by then)
// stores the new value and thereby clears the counter.  Call from one thread per head, after a
// __syncthreads() that follows the head's last global write.
// FENCED: for readers inside the same kernel, who take the new value as the sign that every head's writes are
// there (each arriving head fences before the call, the last one again before it stores).
template <bool FENCED = false>
__device__ __forceinline__ void arrive_and_set(int32_t *win_pos, int b, int heads_v, int new_value) {
  const int old = atomicAdd(win_pos + b, 0x10000);
  if ((old >> 16) == heads_v - 1) {
    if (FENCED) __threadfence();
    win_pos[b] = new_value;
  }
}

}  // namespace lq
