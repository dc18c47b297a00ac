// One decode step as ONE kernel: the decode of all heads and the window boundaries of the sequences whose window
// fills with this token run side by side (Sec. 3.3: the boundary work is meant to hide under the state stream).
//
// The decode is bound by the memory system, the boundary by the fp32 pipes; as two kernels one after the other
// each leaves the other resource idle.  Here every SM holds two CTAs of 256 threads: a DECODE CTA, three
// independent pairs of warps with a shared-memory slot each (decode_slot of lq_decode.cuh), and a BOUNDARY CTA,
// which holds one 128x128 state in registers (reconstruct_tile, quantize_tile of lq_boundary.cuh).
//
// Order of work: the decode slots first take the heads that sit at their last free record (their window fills
// with this token), then all others.  A boundary CTA owns heads f, f + F, f + 2F, ... (F boundary CTAs); it looks
// at their sequences' win_pos until one reads W - which the last of the sequence's heads to be decoded stores,
// after the writes of all of them - takes that head through the boundary, and leaves when every decode slot has
// reported the end of its first pass and nothing of its own is left.  The decode never waits for a boundary CTA,
// a boundary CTA waits only for decode work, and the kernel is launched cooperatively (all CTAs resident), so the
// waiting cannot deadlock; it is bounded all the same, and gives up with an error flag.
#pragma once
#include "lq_boundary.cuh"
#include "lq_decode.cuh"

namespace lq {

constexpr int FUSED_SLOTS = 3;               // decode slots (pairs of warps) per decode CTA
constexpr int FUSED_NBUF = 256;              // window positions a slot can hold: its number of heads is at most this

// bytes of dynamic shared memory: the larger of the two kinds of CTA
inline size_t fused_smem_bytes(int W, int r, bool diag, bool rec16) {
  const size_t dec = (size_t)FUSED_SLOTS * (DecodeSlot(W, r, diag, rec16).bytes + 2 * FUSED_NBUF);
  const size_t bnd = BoundarySmem::bytes(W, r, diag, rec16, 1);
  return dec > bnd ? dec : bnd;
}

// One head through the window boundary (the body of boundary_kernel's loop, single staging buffer).  The data
// was written by other SMs during this kernel: everything is fetched through the L2.
template <int GATE, bool R16>
__device__ __forceinline__ void fused_boundary_head(const Params &p, float *smem, const Tile &t, size_t bh, int n) {
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  const BoundarySmem sm(smem, p.W, p.r, DIAG, R16, 0);
  const int b = static_cast<int>(bh / p.heads_v);
  float M[8][8];
  stage_issue<GATE, R16>(p, sm, t, bh, n);
  cp_async_commit();
  cp_async_wait_all();
  // (the 4-byte copies of the scalar gate's decays go through the L1, which may hold an older copy of the line)
  if (!DIAG && t.tid < n) sm.ba[t.tid] = __ldcg(p.decays + bh * (size_t)p.W + t.tid);
  __syncthreads();
  reconstruct_tile<GATE, R16>(p, sm, t, bh, n, M);
  quantize_tile<MAX_R>(p, sm, t, bh, n, M);
  __syncthreads();                           // this head's use of shared memory is over
  if (t.tid == 0) arrive_and_set(p.win_pos, b, p.heads_v, 0);
}

template <int GATE, bool R16>
__device__ __forceinline__ void fused_boundary_role(const Params &p, float *smem, const unsigned f, const unsigned F,
                                                    const unsigned decode_slots) {
  const Tile t;
  const size_t nh = (size_t)p.batch * p.heads_v;
  __shared__ uint32_t done_mask[64];         // one bit per own head: taken through the boundary
  __shared__ uint32_t ready_mask;
  __shared__ int finished;
  const unsigned own = f < nh ? static_cast<unsigned>((nh - 1 - f) / F + 1) : 0;     // heads f + k F, k < own
  for (int i = t.tid; i < 64; i += 256) done_mask[i] = 0;
  if (t.tid == 0) finished = 0;
  __syncthreads();
  if (own > 64 * 32) {                       // more heads than the bit mask holds (the host does not launch this)
    if (t.tid == 0) atomicOr(&g_device_error, 4);
    return;
  }
  bool last_sweep = false;                   // the decode slots are through with their first pass: one more look
  for (unsigned spin = 0;; spin++) {
    bool any = false;
    for (unsigned k0 = 0; k0 < own; k0 += 32) {
      if (t.warp == 0) {
        const unsigned k = k0 + t.lane;
        bool ready = false;
        if (k < own && !((done_mask[k >> 5] >> (k & 31)) & 1u)) {
          const size_t bh = f + (size_t)k * F;
          const int x = *reinterpret_cast<volatile const int *>(p.win_pos + bh / p.heads_v);
          ready = (x & 0xFFFF) == p.W;       // stored by the sequence's last head, after every head's writes
        }
        const uint32_t m = __ballot_sync(FULL, ready);
        if (t.lane == 0) ready_mask = m;
      }
      __syncthreads();
      uint32_t m = ready_mask;
      __syncthreads();                       // ready_mask is rewritten by the next group
      if (m) __threadfence();                // what the arrivals published is read after this
      while (m) {
        const int kbit = __ffs(m) - 1;
        m &= m - 1;
        const unsigned k = k0 + kbit;
        fused_boundary_head<GATE, R16>(p, smem, t, f + (size_t)k * F, p.W);
        if (t.tid == 0) done_mask[k >> 5] |= 1u << (k & 31);
        __syncthreads();
        any = true;
      }
    }
    if (any) continue;
    if (last_sweep) break;
    if (t.tid == 0) {
      const unsigned d = *reinterpret_cast<volatile unsigned *>(&g_fused_boundary_heads_done);
      finished = d >= decode_slots || spin > (1u << 18);
      if (spin > (1u << 18)) atomicOr(&g_device_error, 2);      // gave up waiting for the decode
    }
    __syncthreads();
    last_sweep = finished != 0;
    __syncthreads();
    if (!last_sweep) __nanosleep(500);
  }
}

template <int GATE, bool R16>
__global__ void __launch_bounds__(256, 2) fused_step_kernel(const Params p, const int decode_ctas) {
  extern __shared__ float4 lq_fused_smem[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(lq_fused_smem);
  const unsigned decode_slots = static_cast<unsigned>(decode_ctas) * FUSED_SLOTS;
  const unsigned parties = decode_slots + (gridDim.x - decode_ctas);     // who takes an exit ticket
  bool ticket = false;
  if (static_cast<int>(blockIdx.x) < decode_ctas) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, s = warp >> 1;
    if (s >= FUSED_SLOTS) return;            // (two warps of the CTA have nothing to do)
    const size_t slot_bytes = DecodeSlot(p.W, p.r, GATE == LQ_GATE_DIAG, R16).bytes + 2 * FUSED_NBUF;
    unsigned char *slot = smem + s * slot_bytes;
    uint16_t *nbuf = reinterpret_cast<uint16_t *>(slot + slot_bytes - 2 * FUSED_NBUF);
    const unsigned first = blockIdx.x * FUSED_SLOTS + s;
    uint32_t parA = 0, parR = 0;
    decode_slot_init<GATE, R16, true>(p, slot, lane, warp & 1, 5 * s, first, decode_slots, nbuf);
    decode_slot<GATE, R16, true, 0>(p, slot, lane, warp & 1, 5 * s, first, decode_slots, nbuf, parA, parR);
    decode_slot<GATE, R16, true, 1>(p, slot, lane, warp & 1, 5 * s, first, decode_slots, nbuf, parA, parR);
    ticket = (warp & 1) == 1 && lane == 0;   // the dot warp is the slot's last word
  } else {
    fused_boundary_role<GATE, R16>(p, reinterpret_cast<float *>(smem), blockIdx.x - decode_ctas,
                                   gridDim.x - decode_ctas, decode_slots);
    ticket = threadIdx.x == 0;
  }
  if (ticket && atomicAdd(&g_fused_exit_ticket, 1u) == parties - 1) {   // the last one out clears the counters
    g_fused_boundary_heads_done = 0;
    g_fused_exit_ticket = 0;
    __threadfence();
  }
}

}  // namespace lq
