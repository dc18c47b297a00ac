// Decode: one token for one (sequence, value head), done by a CTA of two warps with different roles.
//
// Eq. 10 (readout of the smoothed, compensated window representation) evaluated for x = alpha.k and
// x = alpha.q in one pass over the 8-bit codes:
//   S_{l-1}^T (alpha.x) = (B/127) Z^T (C Gamma_{1:l} x) + Uc (Kc^T Gamma_{1:l} x) + sum_j u_j (kt_j^T Gamma_{j+1:l} x)
// then u = v - S_{l-1}^T(alpha.k) (Eq. 3), o = S_{l-1}^T(alpha.q) + u (kt^T q), and the record is appended.
//
// Data movement: a head's block (16 KiB of codes, the two scale vectors, the compensators: 19 KiB) and
// its n buffered record rows are each contiguous in memory and are brought into the CTA's shared-memory slot
// by TWO TMA bulk copies, each completing on its own mbarrier: a few large bulk requests keep the memory
// system busy where thousands of 16-byte loads could not (plain loads are limited per warp), and about 64 KB
// in flight per SM saturate HBM.  The slot is small enough for six CTAs per SM.  CTAs are persistent and walk
// over the heads with a grid stride.  No load sits on a head's critical path (with the memory system kept
// full a load takes microseconds to return): the token's vectors are loaded into registers one head ahead,
// the per-head scalars (window position, beta, scalar alpha) for 32 heads at a time, one per lane; whatever
// needs only the token (the scalar-gate decay chain, kt^T q) is computed before the wait for the slot.
//
// Roles: the STREAM warp turns C Gamma x into fixed-point digits, runs the tensor-core pass over the codes,
// adds the compensator terms, requests the next head's block as soon as nobody needs this one's any more,
// adds the record terms and finishes u and o; the DOT warp meanwhile projects onto the compensators, walks
// the buffered records (projections and the records' terms of the readout in one pass), requests the next
// head's records, appends the new record and makes the window-position arrival.  They meet at named barriers
// (three per head, four with the diagonal gate, whose decays both warps read from the records).
//
// Arithmetic: the first term is a dense int8 contraction, Z^T [128 x 128] against the two vectors.  The
// vectors are put on a 30-bit block fixed-point grid and split into four signed base-256 digits each, which
// gives an int8 operand of 128 x 8; the tensor cores (mma.sync m16n8k32, s8 x s8 -> s32) produce exact
// integer sums, recombined in 64-bit integers and rounded to fp32 once, so the result does not depend on
// the order of accumulation.  The codes are stored value-channel major (Z^T, [d_v][d_k]): the contraction
// index is then contiguous, as the MMA operand layout needs.  The small dot products against records and
// compensators run on the fp32 pipes in the library's fixed summation order.
#pragma once
#include <type_traits>

#include "lq_common.cuh"

namespace lq {

// Set when a bounded wait gave up (bit 0: a decode warp's wait for one of its bulk copies; bits 1, 2: the fused step
// kernel's waits; bit 3: the wait of lq_selftest_bounded_wait).  Never cleared by kernels: lq_clear_device_flags.
__device__ int g_device_error = 0;

// Rows of the record buffer that a decode slot holds at a time (a multiple of four: the walk takes the records four
// at a time from the newest back, so a group of four never straddles two segments).
constexpr int REC_SEG = 32;                // (16 was tried: no faster at W = 32 or 64)

// ---- shared-memory slot of one CTA ----
struct DecodeSlot {
  // byte offsets inside the slot; every region starts on a 16-byte boundary
  int head, rec, bas, digits, y, pk, pq, mbar, bytes;
  __host__ __device__ DecodeSlot(int W, int r, bool diag, bool rec16 = false) {
    // a window holds at most W-1 records when a token arrives; they are staged REC_SEG rows at a time (newest
    // first), which keeps the slot small for long windows
    int rows = W > 1 ? W - 1 : 1;
    if (rows > REC_SEG) rows = REC_SEG;
    int o = 0;
    head = o; o += head_bytes(r);          // the head block: codes | col_scale | row_smooth | comp_k | comp_u
    rec = o; o += (rec16 ? 2 : 4) * record_floats(diag) * rows;   // buffered record rows (fp32 or fp16)
    bas = o; o += diag ? 0 : 2 * 4 * MAX_W;         // scalar gate: the records' decays, one copy per warp
    digits = o; o += 8 * D;               // digit planes: plane 4v+d = digit d of vector v (0: k, 1: q)
    y = o; o += 2 * 4 * D;                // [2][128]: the rounded sums of the state stream, later the record terms
    pk = o; o += (4 * (r + 2) + 15) / 16 * 16;      // compensator projections against Gamma k
    pq = o; o += (4 * (r + 2) + 15) / 16 * 16;      // ... against Gamma q; pq[r], pq[r+1] hold kt^T q of alternate heads
    mbar = o; o += 16;
    bytes = (o + 127) / 128 * 128;
  }
};

// D(16x8, s32) += A(16x32, s8, row-major) * B(32x8, s8, column-major)
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
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
// The arrival that announces the bytes of the next copies.  Relaxed: nothing this thread wrote has to be
// visible to anybody through this barrier (the copies' own completion is what the waiters acquire), and the
// default release form stalls the warp for about 800 cycles here.
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.relaxed.cta.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> shared bulk copy; addresses and size are multiples of 16 bytes
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// The same with an L2 eviction priority for the lines the copy brings in.
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
// Ask the L2 for a piece of global memory (no data comes back, nothing waits for it).
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(src), "r"(bytes) : "memory");
}
// Bounded wait for phase `parity`; false if the limit of LIMIT polls ran out (the caller then reports and bails out).
template <int LIMIT = (1 << 20)>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int spin = 0; spin < LIMIT; spin++) {
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

// sums of four values over sixteen neighbouring lanes each, the four shuffle chains interleaved
__device__ __forceinline__ void tree16x4(float (&x)[4]) {
#pragma unroll
  for (int s = 1; s <= 8; s <<= 1) {
#pragma unroll
    for (int v = 0; v < 4; v++) x[v] = x[v] + __shfl_xor_sync(FULL, x[v], s);
  }
}

// Named barriers of the CTA (64 threads each): one side arrives, the other waits.
//   1: dot warp -> stream warp, "the projections are in shared memory"
//   2: stream warp -> dot warp, "the slot may be overwritten"
__device__ __forceinline__ void named_arrive(int id) {
  __threadfence_block();
  asm volatile("bar.arrive %0, 64;\n" ::"r"(id) : "memory");
}
__device__ __forceinline__ void named_wait(int id) { asm volatile("bar.sync %0, 64;\n" ::"r"(id) : "memory"); }

// The token's vectors as raw bf16 bits, loaded one head ahead: lane c (and its twin c+16) owns key
// channels 8c..8c+7, lane l value channels 4l..4l+3.
struct TokenRaw {
  uint4 k, q, a;        // a: diagonal-gate alpha
  uint2 v;
  float ba_lo, ba_hi;   // scalar gate: decays of buffered records `lane` and `lane + 32` (stale beyond n)
};

// A head index with its sequence and value-head parts, stepped without divisions.
struct HeadIdx {
  unsigned bh, b, hv;
  __device__ __forceinline__ void step(unsigned dbh, unsigned db, unsigned dhv, unsigned heads_v) {
    bh += dbh; b += db; hv += dhv;
    if (hv >= heads_v) { hv -= heads_v; b += 1; }
  }
};

template <int GATE>
__device__ __forceinline__ void load_token(const Params &p, const HeadIdx h, int group, int lane, int role, TokenRaw &tk) {
  const int c = lane & 15;
  const size_t bh = h.bh;
  const size_t qk_off = ((size_t)h.b * p.heads_qk + h.hv / group) * D;
  tk.k = *reinterpret_cast<const uint4 *>(p.k + qk_off + 8 * c);
  tk.q = *reinterpret_cast<const uint4 *>(p.q + qk_off + 8 * c);
  if (role == 0) tk.v = *reinterpret_cast<const uint2 *>(p.v + bh * D + 4 * lane);
  if (GATE == LQ_GATE_DIAG) {
    tk.a = *reinterpret_cast<const uint4 *>(p.alpha + bh * D + 8 * c);
  } else {
    if (lane < p.W) tk.ba_lo = p.decays[bh * (size_t)p.W + lane];
    if (lane + 32 < p.W) tk.ba_hi = p.decays[bh * (size_t)p.W + lane + 32];
  }
}

// Counters of the fused step kernel (lq_fused.cuh): decode slots that are through with the heads whose window
// becomes full, and CTAs that have left; the last CTA to leave clears both.
__device__ unsigned g_fused_boundary_heads_done = 0, g_fused_exit_ticket = 0;

// The work of one pair of warps (role 0: stream warp, role 1: dot warp) on its shared-memory slot: heads
// first, first + G, first + 2G, ...  The named barriers it uses are bar0 + 1 .. bar0 + 5.
// FUSED (the step kernel that also takes the window boundaries): two passes over the heads, first those whose
// window becomes full with this token, so that their boundaries can start while the rest is decoded; the
// arrival on win_pos comes after BOTH warps' global writes of the head, because another CTA acts on it;
// and the window positions of all of the slot's heads are read once, up front, into nbuf (a sequence whose
// boundary is taken meanwhile goes back to position 0, which must not be mistaken for a fresh window).
// Before the first pass: the slot's two copy barriers, and (fused) the window positions of all its heads.
template <int GATE, bool R16, bool FUSED>
__device__ __forceinline__ void decode_slot_init(const Params &p, unsigned char *slot, const int lane, const int role,
                                                 const int bar0, const unsigned first, const unsigned G, uint16_t *nbuf) {
  const DecodeSlot L(p.W, p.r, GATE == LQ_GATE_DIAG, R16);
  const uint32_t barA = smem_addr(slot + L.mbar), barR = barA + 8;
  if (role == 0 && lane == 0) { mbar_init(barA, 1); mbar_init(barR, 1); }
  if (FUSED) {
    const unsigned nh = static_cast<unsigned>(p.batch) * p.heads_v;
    for (unsigned k = 32 * role + lane; first + k * G < nh; k += 64)
      nbuf[k] = static_cast<uint16_t>(p.win_pos[(first + k * G) / p.heads_v] & 0xFFFF);
  }
  named_wait(bar0 + 1);                      // both warps: the barriers are initialised, nbuf is complete
}

// PASS: 0 in the ordinary kernel; in the fused one 0 = the heads whose window fills with this token, 1 = the
// others (two instances of the code: only the first carries the fences that publish a head to other CTAs, and a
// fence anywhere in the loop costs every trip).  parA, parR: the phases of the two copy barriers, carried over.
// LONGW: the window may hold more records than the slot stages at a time (W - 1 > REC_SEG); in the instances for
// shorter windows everything to do with a second segment drops out at compile time.
template <int GATE, bool R16, bool FUSED, int PASS, bool LONGW = true>
__device__ __forceinline__ void decode_slot(const Params &p, unsigned char *slot, const int lane, const int role,
                                            const int bar0, const unsigned first, const unsigned G,
                                            uint16_t *nbuf, uint32_t &parA, uint32_t &parR) {
  constexpr int pass = PASS;
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  constexpr int RF = record_floats(DIAG);
  const int W = p.W, r = p.r;
  using rec_t = typename std::conditional<R16, __half, float>::type;   // element type of the record rows
  const DecodeSlot L(W, r, DIAG, R16);
  const int c = lane & 15, half = lane >> 4, g = lane >> 2, t = lane & 3;
  const int8_t *zt = reinterpret_cast<const int8_t *>(slot + L.head + HB_CODES);
  const float *bs = reinterpret_cast<const float *>(slot + L.head + HB_COL_SCALE);
  const float *cs = reinterpret_cast<const float *>(slot + L.head + HB_ROW_SMOOTH);
  const uint16_t *ckh = reinterpret_cast<const uint16_t *>(slot + L.head + HB_COMP_K);
  const uint16_t *cuh = reinterpret_cast<const uint16_t *>(slot + L.head + hb_comp_u(r));
  const rec_t *rec = reinterpret_cast<const rec_t *>(slot + L.rec);     // rows of RF elements: kt | u | (alpha)
  float *bas = reinterpret_cast<float *>(slot + L.bas) + role * MAX_W;   // this warp's copy of the decays
  int8_t *digits = reinterpret_cast<int8_t *>(slot + L.digits);
  float *y = reinterpret_cast<float *>(slot + L.y), *pk = reinterpret_cast<float *>(slot + L.pk);
  float *pq = reinterpret_cast<float *>(slot + L.pq);
  const uint32_t barA = smem_addr(slot + L.mbar), barR = barA + 8, slot_a = smem_addr(slot);   // head block, records

  const unsigned nh = static_cast<unsigned>(p.batch) * p.heads_v, Hv = p.heads_v;
  const unsigned G_b = G / Hv, G_hv = G % Hv;       // one grid stride in (sequence, head) steps
  const int group = p.heads_v / p.heads_qk;

#ifdef LQ_TIMING
  long long tick_ = clock64();
  unsigned acc_[12] = {0};
#endif
  // The slot is filled by two bulk copies with a barrier each, because its two parts become free at different
  // times.  The head block (codes, scales, compensators) of the next head is requested by the stream warp as soon
  // as both warps have taken the last thing they need from it (the compensator rows), the records by the dot
  // warp as soon as it has walked them: about half of a head's work later the wait for the next head starts, and
  // by then the copies have been on their way for a while.
  // The regions the copies overwrite were only READ through ordinary loads, whose values have been used
  // before the call; the warps write only their scratch regions.  So nothing written by the generic proxy is
  // at stake and no cross-proxy fence is needed (it costs over a thousand cycles here).
  // A head at its last free record (n == W - 1) goes through the window boundary right after this kernel, which
  // reads the same head block and records again: its lines are asked to stay in the L2 until then.
  const uint64_t keep = l2_keep_policy(), stream = l2_stream_policy();
  auto request_head = [&](unsigned bh, int n) {
    if (lane == 0) {
      mbar_expect_tx(barA, head_bytes(r));
      if (n == W - 1) bulk_g2s_hint(slot_a + L.head, p.head(bh), head_bytes(r), barA, keep);
      else bulk_g2s_hint(slot_a + L.head, p.head(bh), head_bytes(r), barA, stream);
    }
  };
  // first record of the segment that ends before record `hi`
  auto seg_base = [&](int hi) { return (LONGW && hi > REC_SEG) ? hi - REC_SEG : 0; };
  // records [seg_base(hi), hi) of head bh, n of which are buffered in all, into the slot
  auto request_segment = [&](unsigned bh, int n, int hi) {
    if (lane == 0) {
      const int lo = seg_base(hi);
      const uint32_t rb = static_cast<uint32_t>(sizeof(rec_t)) * RF * (hi - lo);
      mbar_expect_tx(barR, rb);              // with no records the phase completes at once
      if (hi > lo) {
        if (n == W - 1) bulk_g2s_hint(slot_a + L.rec, p.record<rec_t>(bh, lo, DIAG), rb, barR, keep);
        else bulk_g2s_hint(slot_a + L.rec, p.record<rec_t>(bh, lo, DIAG), rb, barR, stream);
      }
    }
  };
  auto request_records = [&](unsigned bh, int n) { request_segment(bh, n, n); };   // the newest segment
  // Bounded wait for one of the two.  A copy that never lands must not hang the GPU: when the limit runs out the
  // error flag is set and the warp goes on (its results are garbage, the flag says so); the other warp, which
  // meets this one at the named barriers, is not left waiting.
  auto wait_for = [&](uint32_t bar_, uint32_t &par) {
    if (!mbar_wait(bar_, par) && lane == 0) atomicOr(&g_device_error, 1);
    par ^= 1u;
    __syncwarp();
  };

  // Equal shares do not take equal time: pairs that share an SM with fewer others, or sit nearer the memory they
  // read, are through with ten heads when others have done eight.  With scratch words in the state (lq_state.work)
  // every pair therefore takes only its first S heads in turn (DRAWN_ROUNDS rounds fewer than would fall to it), and
  // the heads that are left (S G + t, t < pool) go to whoever gets there first: from its last turn but one on, the dot
  // warp draws a ticket t in every trip, for the head two trips on (word 0 of the scratch words counts the tickets;
  // the boundary kernel behind this one puts it back to zero), hands it to the stream warp with the record terms
  // (barrier 1), and at the end of the trip both warps ask for that head's scalars, which they look at for the first
  // time half a trip later (ext_*) and move to the lane registers of the other heads' at the end of the next trip.
  // A pair stops when a ticket is beyond the pool.
  const int rounds_all = static_cast<int>(nh / G);             // rounds in which every pair has a head
  const int DRAWN_ROUNDS = rounds_all >= 6 ? 2 : 1;            // (with few rounds, more of them in turn)
  const bool draw = !FUSED && p.work != nullptr && rounds_all >= 3;
  const int S = draw ? rounds_all - DRAWN_ROUNDS : 0;
  const unsigned pool = draw ? nh - static_cast<unsigned>(S) * G : 0;
  // Per-head scalars of this CTA's heads, 32 heads at a time: lane l holds those of the CTA's (32*batch+l)-th head
  int sc_n = 0;
  uint32_t sc_beta = 0, sc_alpha = 0;
  auto load_scalars = [&](unsigned first_bh) {
    const unsigned bh = first_bh + lane * G;  // (once per 32 heads: a division is fine here)
    if (bh < (draw ? static_cast<unsigned>(S) * G : nh)) {     // (the heads taken in turn)
      sc_n = FUSED ? nbuf[(first_bh - first) / G + lane]
                   : p.win_pos[bh / Hv];    // bits 16.. are the arrival counter of this launch: masked at use
      sc_beta = p.beta[bh];
      if (!DIAG) sc_alpha = p.alpha[bh];
    }
  };

  // Arrival on win_pos (see arrive_and_set): the counter says how many heads of the sequence have READ the old
  // value, which this head did when its scalars were loaded.  The dot warp makes the arrival, at the end of its
  // work: it has slack, the stream warp (the longer of the two) has none to sit out the atomic's round trip.
  // A head whose window is already full (n >= W) gets no token: it is neither requested nor waited for.
  // which heads this pass takes: all that get a token, or (fused) those at / not at their last free record
  auto wanted = [&](int n_) { return n_ < W && (!FUSED || (n_ == W - 1) == (pass == 0)); };
  load_scalars(first);
  TokenRaw nxt;                               // the token of the head about to start
  nxt.ba_lo = nxt.ba_hi = 1.0f;
  HeadIdx hd{first, first / Hv, first % Hv};  // this head and the next one
  HeadIdx hd1 = hd;
  hd1.step(G, G_b, G_hv, Hv);
  {
    const int n0 = __shfl_sync(FULL, sc_n, 0) & 0xFFFF;
    if (first < nh && wanted(n0)) {
      load_token<GATE>(p, hd, group, lane, role, nxt);
      if (role == 0) request_head(first, n0);
      else request_records(first, n0);
    }
  }
#ifdef LQ_TIMING
  tick_ = clock64();
#endif
  unsigned *qidx = reinterpret_cast<unsigned *>(pk + r);      // (a spare word of the projection area)
  unsigned ticket = 0xFFFFFFFFu;             // (dot warp, lane 0) what was drawn in this trip
  bool drawing = draw;                       // no ticket has been beyond the pool yet
  int ext_n = 0;                             // scalars of the head drawn a trip ago, on their way
  uint32_t ext_beta = 0, ext_alpha = 0;
  int idx = 0;                               // position of the head in this slot's list
  // end of a trip
  auto finish_trip = [&]() {
    // the next head, if it was drawn: its scalars, asked for a trip ago, go where the others' are
    if (draw && idx + 1 >= S && lane == ((idx + 1) & 31)) { sc_n = ext_n; sc_beta = ext_beta; sc_alpha = ext_alpha; }
    unsigned extra = nh;                     // the head after the next one, if it is a drawn one
    if (drawing && idx + 2 >= S) {
      const unsigned tk = role == 1 ? __shfl_sync(FULL, ticket, 0) : *reinterpret_cast<volatile unsigned *>(qidx);
      if (tk < pool) {
        extra = static_cast<unsigned>(S) * G + tk;
        ext_n = p.win_pos[extra / Hv];
        ext_beta = p.beta[extra];
        if (!DIAG) ext_alpha = p.alpha[extra];
      } else {
        drawing = false;
      }
    }
    hd = hd1;
    idx++;
    if (!draw || idx + 1 < S) {
      hd1.step(G, G_b, G_hv, Hv);
    } else if (extra < nh) {
      const unsigned b_ = extra / Hv;
      hd1 = HeadIdx{extra, b_, extra - b_ * Hv};
    } else {
      hd1 = HeadIdx{nh, 0u, 0u};
    }
  };
  for (; hd.bh < nh; finish_trip()) {
    const bool draws = drawing && idx + 2 >= S;                 // a ticket is drawn in this trip
    if (draws && role == 1 && lane == 0) ticket = static_cast<unsigned>(atomicAdd(p.work, 1));
    const size_t bh = hd.bh;
    const int n = __shfl_sync(FULL, sc_n, idx & 31) & 0xFFFF;
    const float beta = __uint_as_float(__shfl_sync(FULL, sc_beta, idx & 31) << 16);
    const float alpha_s = __uint_as_float(__shfl_sync(FULL, sc_alpha, idx & 31) << 16);
    // the next head's scalars: from the next batch when this head is the last of its batch
    const unsigned bh_next = hd1.bh;
    if ((idx & 31) == 31) load_scalars(bh_next);
    // The next head's window position.  Of a drawn head it is still on its way (ext_n, asked for at the end of the
    // trip before): it is looked at only where the head's data is requested, half a trip from here; until then the
    // head counts as one that gets a token (its token is loaded, which does no harm if it gets none).
    const bool next_drawn = draw && idx + 1 >= S;
    const int n_next_turn = bh_next < nh ? (__shfl_sync(FULL, sc_n, (idx + 1) & 31) & 0xFFFF) : W;
    auto n_next_now = [&]() { return next_drawn ? (bh_next < nh ? (ext_n & 0xFFFF) : W) : n_next_turn; };
    const bool next_token = next_drawn ? bh_next < nh : wanted(n_next_turn);
    const bool active = wanted(n);
    const int b = static_cast<int>(hd.b);
    LQ_TICK(0);

    if (!active) {                           // nothing was requested for this head; keep the pipeline going
      const int n_next = n_next_now();
      if (wanted(n_next)) {
        load_token<GATE>(p, hd1, group, lane, role, nxt);
        if (role == 0) request_head(bh_next, n_next);
        else request_records(bh_next, n_next);
      }
      if (draws) {                           // the ticket changes hands outside the usual place
        if (role == 1) {
          if (lane == 0) *qidx = ticket;
          __syncwarp();
          named_arrive(bar0 + 1);
        } else {
          named_wait(bar0 + 1);
        }
      }
      continue;
    }

    // ---- this head's token (loaded while the previous head was being worked on); once it is unpacked
    // the registers are free for the next head's, whose load is then issued ----
    float k8[8], q8[8], a8[8];
    widen8_bf16(nxt.k, k8);
    widen8_bf16(nxt.q, q8);
    const uint2 v_raw = nxt.v;
    if (DIAG) {
      widen8_bf16(nxt.a, a8);
    } else {
#pragma unroll
      for (int e = 0; e < 8; e++) a8[e] = alpha_s;
      bas[lane] = nxt.ba_lo;
      bas[lane + 32] = nxt.ba_hi;
    }
    if (next_token) load_token<GATE>(p, hd1, group, lane, role, nxt);        // used one trip from now
    // scalar gate: Gamma_{1:l}, the chain of decays from the newest record back (Appendix B.2), needs nothing
    // from the slot, so the stream warp takes it before it waits
    float gsc = alpha_s;
    if (!DIAG) {
      __syncwarp();
#pragma unroll 4
      for (int j = n - 1; j >= 0; j--) gsc = gsc * bas[j];
    }
    // kt^T q needs only the token: the dot warp takes it before the wait as well.  It goes to one of two places
    // in turn, because the stream warp may still be reading the previous head's.
    if (role == 1) {
      float2 k2p[4], q2p[4];
#pragma unroll
      for (int cc = 0; cc < 4; cc++) {
        k2p[cc] = __fmul2_rn(pair(beta), make_float2(k8[2 * cc], k8[2 * cc + 1]));
        q2p[cc] = make_float2(q8[2 * cc], q8[2 * cc + 1]);
      }
      const float ktq_pre = tree16(block8(k2p, q2p));
      if (lane == 0) pq[r + (idx & 1)] = ktq_pre;
    }
    LQ_TICK(1);

    // ---- the stream warp waits for the head block; the dot warp first takes the records, which it asked for
    // earlier and which need nothing from the head block, and waits for the block when it gets to the compensators ----
    if (role == 0 && !DIAG) wait_for(barA, parA);  // (diagonal gate: after its own walk of the records' decays)
    LQ_TICK(2);
    if (idx == 0) LQ_STAMP(0, 2);

    if (role == 1) {
      // =========================== DOT WARP ===========================
      // Projections.  A dot product of 128 terms is taken by sixteen lanes (lane c owns block c of eight
      // terms); the two halves of the warp work on different vectors, two per half and trip, so that four
      // shuffle trees overlap.  Both halves make the same number of trips (the shuffles name all 32 lanes);
      // an index outside the range recomputes a valid item and is not stored.
      // Records are walked from the newest back, with g8 = Gamma_{j+1:l} kept up on the way (Appendix B.2).
      float2 k2[4], q2[4], a2[4], g2[4], kt2[4];
#pragma unroll
      for (int cc = 0; cc < 4; cc++) {
        k2[cc] = make_float2(k8[2 * cc], k8[2 * cc + 1]);
        q2[cc] = make_float2(q8[2 * cc], q8[2 * cc + 1]);
        a2[cc] = make_float2(a8[2 * cc], a8[2 * cc + 1]);
        g2[cc] = a2[cc];
        kt2[cc] = __fmul2_rn(pair(beta), k2[cc]);
      }
      wait_for(barR, parR);                  // the newest segment of the records
      // Compensator keys against Gamma_{1:l} k and Gamma_{1:l} q (the projections go to pk[h], pq[h]).
      auto project_compensators = [&](const float2 (&gam)[4]) {
        float2 gk2[4], gq2[4];
#pragma unroll
        for (int cc = 0; cc < 4; cc++) { gk2[cc] = __fmul2_rn(gam[cc], k2[cc]); gq2[cc] = __fmul2_rn(gam[cc], q2[cc]); }
        for (int hb = 0; hb < r; hb += 4) {
          float s4[4];
          int ho[2];
#pragma unroll
          for (int u = 0; u < 2; u++) {
            ho[u] = hb + 2 * u + half;
            const int h = ho[u] < r ? ho[u] : r - 1;
            float x8[8];
            widen8_f16(*reinterpret_cast<const uint4 *>(ckh + h * D + 8 * c), x8);
            float2 x2[4];
#pragma unroll
            for (int cc = 0; cc < 4; cc++) x2[cc] = make_float2(x8[2 * cc], x8[2 * cc + 1]);
            s4[2 * u] = block8(x2, gk2);
            s4[2 * u + 1] = block8(x2, gq2);
          }
          tree16x4(s4);
#pragma unroll
          for (int u = 0; u < 2; u++)
            if (c == 0 && ho[u] < r) { pk[ho[u]] = s4[2 * u]; pq[ho[u]] = s4[2 * u + 1]; }
        }
      };
      float rk_rec[4] = {0.0f, 0.0f, 0.0f, 0.0f}, rq_rec[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      int base = seg_base(n);                        // the slot holds records base .. (row = record - base)
      for (int jt = n - 1; jt >= 0; jt -= 4) {       // records jt, jt-1, jt-2, jt-3
        if (LONGW && jt < base) {                    // the segment is walked: fetch the one before it
          __syncwarp();
          if (DIAG) named_wait(bar0 + 4);            // (the stream warp has taken this segment's decays as well)
          request_segment(bh, n, base);
          base = seg_base(base);
          wait_for(barR, parR);
        }
        float s4[4];
        int jo[2];
#pragma unroll
        for (int u = 0; u < 2; u++) {
          // the decays of the two records of this pair; the half that owns the older one steps over the newer
          const int jn = jt - 2 * u, jold = jn - 1;  // newer, older
          float2 an[4], ao[4], gmine[4];
          if (DIAG) {
            load8p(rec + ((jn > 0 ? jn : 0) - base) * RF + REC_A + 8 * c, an);
            load8p(rec + ((jold > 0 ? jold : 0) - base) * RF + REC_A + 8 * c, ao);
          } else {
            const float2 x = pair(bas[jn > 0 ? jn : 0]), z = pair(bas[jold > 0 ? jold : 0]);
#pragma unroll
            for (int cc = 0; cc < 4; cc++) { an[cc] = x; ao[cc] = z; }
          }
#pragma unroll
          for (int cc = 0; cc < 4; cc++) {
            const float2 gn = g2[cc], go = __fmul2_rn(gn, an[cc]);   // Gamma_{jn+1:l}, Gamma_{jold+1:l}
            gmine[cc] = half ? go : gn;
            // past both records; the chain stops at record 0, so that it ends as Gamma_{1:l} exactly
            // (selects: a branch for the last trip of a long head was slower)
            g2[cc] = (!DIAG || jold >= 0) ? __fmul2_rn(go, ao[cc]) : (jn >= 0 ? go : gn);
          }
          jo[u] = jn - half;
          const int j = jo[u] >= 0 ? jo[u] : 0;      // (record 0 is in the slot whenever an index runs below it)
          float2 x2[4], yk2[4], yq2[4];
          load8p(rec + (j - base) * RF + REC_KT + 8 * c, x2);
#pragma unroll
          for (int cc = 0; cc < 4; cc++) { yk2[cc] = __fmul2_rn(gmine[cc], k2[cc]); yq2[cc] = __fmul2_rn(gmine[cc], q2[cc]); }
          s4[2 * u] = block8(x2, yk2);
          s4[2 * u + 1] = block8(x2, yq2);
        }
        tree16x4(s4);
        // The record terms sum_j u_j (kt_j^T Gamma k) and the same for q, channels 4 lane .. 4 lane + 3, as one
        // chain from the newest record back.  Half 0 holds the projections of records jt and jt-2, half 1
        // those of jt-1 and jt-3: swap them, then take the four records in order.
        {
          float oth[4];
#pragma unroll
          for (int e = 0; e < 4; e++) oth[e] = __shfl_xor_sync(FULL, s4[e], 16);
#pragma unroll
          for (int i4 = 0; i4 < 4; i4++) {
            const int j = jt - i4;
            if (j < 0) break;                                  // the same for every lane
            const int u = i4 >> 1;
            const bool mine = (i4 & 1) == half;
            const float pkj = mine ? s4[2 * u] : oth[2 * u], pqj = mine ? s4[2 * u + 1] : oth[2 * u + 1];
            const float4 u4 = load4(rec + (j - base) * RF + REC_U + 4 * lane);
            rk_rec[0] = fmaf(u4.x, pkj, rk_rec[0]); rq_rec[0] = fmaf(u4.x, pqj, rq_rec[0]);
            rk_rec[1] = fmaf(u4.y, pkj, rk_rec[1]); rq_rec[1] = fmaf(u4.y, pqj, rq_rec[1]);
            rk_rec[2] = fmaf(u4.z, pkj, rk_rec[2]); rq_rec[2] = fmaf(u4.z, pqj, rq_rec[2]);
            rk_rec[3] = fmaf(u4.w, pkj, rk_rec[3]); rq_rec[3] = fmaf(u4.w, pqj, rq_rec[3]);
          }
        }
      }
      LQ_TICK(3);
      // Now the head block: the compensators are projected with Gamma_{1:l}, which for the diagonal gate is where
      // the walk's chain of decays has arrived (g2), for the scalar gate the product taken before the wait.
      wait_for(barA, parA);
      if (r > 0) {
        if (DIAG) {
          project_compensators(g2);
        } else {
          float2 gam[4];
#pragma unroll
          for (int cc = 0; cc < 4; cc++) gam[cc] = pair(gsc);
          project_compensators(gam);
        }
      }
      __syncwarp();
      named_arrive(bar0 + 3);                       // the compensator projections are in pk, pq; this warp is done with the head block
      LQ_TICK(4);
      if (DIAG) named_wait(bar0 + 4);               // diagonal gate: the stream warp read the records' decays too
      {
        const int n_next = n_next_now();
        if (wanted(n_next)) request_records(bh_next, n_next);
      }
      named_wait(bar0 + 2);                         // the stream warp has taken its sums out of y
      *reinterpret_cast<float4 *>(y + 4 * lane) = make_float4(rk_rec[0], rk_rec[1], rk_rec[2], rk_rec[3]);
      *reinterpret_cast<float4 *>(y + D + 4 * lane) = make_float4(rq_rec[0], rq_rec[1], rq_rec[2], rq_rec[3]);
      if (draws && lane == 0) *qidx = ticket;
      __syncwarp();
      named_arrive(bar0 + 1);                       // the record terms are in shared memory (and the ticket)
      LQ_TICK(5);
      // append the key side of the record (and its decay)
      {
        rec_t *row = p.record<rec_t>(bh, n, DIAG);
        if (half == 0) {
          store8p(row + REC_KT + 8 * c, kt2);
          if (DIAG) store8(row + REC_A + 8 * c, a8);
          else if (lane == 0) p.decays[bh * (size_t)W + n] = a8[0];
        }
      }
      if (FUSED && pass == 0) {              // a boundary CTA will read this head's record: the stream warp's u is
        named_wait(bar0 + 5);                // out as well, and both warps' writes are ordered before the arrival
        __threadfence();
      }
      if (lane == 0) arrive_and_set<FUSED && PASS == 0>(p.win_pos, b, p.heads_v, n + 1);
      LQ_TICK(7);
    } else {
      // =========================== STREAM WARP ===========================
      // Gamma_{1:l}: the chain of decays from the newest record back (Appendix B.2)
      float gam[8];
#pragma unroll
      for (int e = 0; e < 8; e++) gam[e] = a8[e];
      if (DIAG) {
        for (int hi = n;;) {                        // segment after segment, in step with the dot warp
          const int lo = seg_base(hi);
          wait_for(barR, parR);
#pragma unroll 2
          for (int j = hi - 1; j >= lo; j--) {
            float aj[8];
            load8(rec + (j - lo) * RF + REC_A + 8 * c, aj);
#pragma unroll
            for (int e = 0; e < 8; e++) gam[e] = gam[e] * aj[e];
          }
          __syncwarp();
          named_arrive(bar0 + 4);                   // this warp is done with the segment
          if (lo == 0) break;
          hi = lo;
        }
        wait_for(barA, parA);
      } else {
#pragma unroll
        for (int e = 0; e < 8; e++) gam[e] = gsc;
      }
      LQ_TICK(3);
      // C Gamma k (lanes 0..15) and C Gamma q (lanes 16..31) on their fixed-point grids, as digit planes
      float back_own;
      {
        float c8[8], x8[8];
        load8(cs + 8 * c, c8);
        float m = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; e++) {
          x8[e] = c8[e] * (gam[e] * (half ? q8[e] : k8[e]));
          m = fmaxf(m, fabsf(x8[e]));
        }
#pragma unroll
        for (int s = 1; s <= 8; s <<= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, s));
        float scale;
        fixed_point_scales(m, scale, back_own);
        // X = d0 + 256 d1 + 65536 d2 + 2^24 d3 with digits in [-128, 127]: the digit is the low byte read as
        // signed, and taking it off is (X + 128) >> 8.  The bytes of the four stages of an element are the
        // four digits; prmt gathers the same digit of four elements into one word.
        uint32_t st[8][4];
#pragma unroll
        for (int e = 0; e < 8; e++) {
          int X = __float2int_rn(x8[e] * scale);
#pragma unroll
          for (int d = 0; d < 4; d++) { st[e][d] = static_cast<uint32_t>(X); X = (X + 128) >> 8; }
        }
#pragma unroll
        for (int d = 0; d < 4; d++) {
          const uint32_t lo = __byte_perm(__byte_perm(st[0][d], st[1][d], 0x0040), __byte_perm(st[2][d], st[3][d], 0x0040), 0x5410);
          const uint32_t hi = __byte_perm(__byte_perm(st[4][d], st[5][d], 0x0040), __byte_perm(st[6][d], st[7][d], 0x0040), 0x5410);
          *reinterpret_cast<uint2 *>(digits + (4 * half + d) * D + 8 * c) = make_uint2(lo, hi);
        }
      }
      const float back_other = __shfl_xor_sync(FULL, back_own, 16);
      const float back_k = half ? back_other : back_own, back_q = half ? back_own : back_other;
      __syncwarp();                          // the digit planes are visible to the warp
      LQ_TICK(4);

      // The state stream on the tensor cores: eight 16-row tiles of Z^T, K = 128 as four k-blocks.  A
      // thread's 16 bytes of a row hold key channels 64p+16t..64p+16t+15 and serve two k-blocks; the digit
      // planes are read with the same permutation of the key index.  The two 64-channel halves of a tile
      // accumulate separately (exact integers: any split gives the same sum), which halves the dependent
      // chain of MMAs.  Digit pairs are recombined in int32 (|sum| < 2^30), the two pairs in int64 (the total has
      // 47 bits), and one rounding takes it to fp32.
      {
        constexpr int h0 = 0, h1 = 64;         // the two 64-channel halves (the same split for every lane)
        const uint4 bfa = *reinterpret_cast<const uint4 *>(digits + g * D + h0 + 16 * t);
        const uint4 bfb = *reinterpret_cast<const uint4 *>(digits + g * D + h1 + 16 * t);
        int pair_lo[8], pair_hi[8];            // digit-pair sums of rows g and g+8 of each tile
#pragma unroll
        for (int mt = 0; mt < 8; mt++) {
          int ca[4] = {0, 0, 0, 0}, cb[4] = {0, 0, 0, 0};
          const int j = 16 * mt + g;
          const uint4 alo = *reinterpret_cast<const uint4 *>(zt + j * D + h0 + 16 * t);
          const uint4 ahi = *reinterpret_cast<const uint4 *>(zt + (j + 8) * D + h0 + 16 * t);
          const uint4 blo = *reinterpret_cast<const uint4 *>(zt + j * D + h1 + 16 * t);
          const uint4 bhi = *reinterpret_cast<const uint4 *>(zt + (j + 8) * D + h1 + 16 * t);
          mma_s8(ca, alo.x, ahi.x, alo.y, ahi.y, bfa.x, bfa.y);
          mma_s8(cb, blo.x, bhi.x, blo.y, bhi.y, bfb.x, bfb.y);
          mma_s8(ca, alo.z, ahi.z, alo.w, ahi.w, bfa.z, bfa.w);
          mma_s8(cb, blo.z, bhi.z, blo.w, bhi.w, bfb.z, bfb.w);
          // c[0], c[1]: row g, planes 2t, 2t+1;  c[2], c[3]: row g+8.  Planes 4v..4v+3 are the digits of
          // vector v: lanes t = 0, 1 carry the k sums and t = 2, 3 the q sums, even t the low digit pair.
          pair_lo[mt] = (ca[0] + cb[0]) + ((ca[1] + cb[1]) << 8);
          pair_hi[mt] = (ca[2] + cb[2]) + ((ca[3] + cb[3]) << 8);
        }
        LQ_TICK(10);
        int oth_lo[8], oth_hi[8];
#pragma unroll
        for (int mt = 0; mt < 8; mt++) {
          oth_lo[mt] = __shfl_xor_sync(FULL, pair_lo[mt], 1);
          oth_hi[mt] = __shfl_xor_sync(FULL, pair_hi[mt], 1);
        }
        if (!(t & 1)) {                      // this lane has the low pairs, its neighbour sent the high pairs
          float *dst = y + (t >> 1) * D + g;
#pragma unroll
          for (int mt = 0; mt < 8; mt++) {
            dst[16 * mt] = __ll2float_rn(static_cast<long long>(oth_lo[mt]) * 65536 + pair_lo[mt]);
            dst[16 * mt + 8] = __ll2float_rn(static_cast<long long>(oth_hi[mt]) * 65536 + pair_hi[mt]);
          }
        }
      }
      __syncwarp();
      LQ_TICK(5);

      // Per value channel (lane l: channels 4l..4l+3): scale the sums, then add the compensator and record
      // terms with the projections of the dot warp
      {
        const float4 yk4 = *reinterpret_cast<const float4 *>(y + 4 * lane);
        const float4 yq4 = *reinterpret_cast<const float4 *>(y + D + 4 * lane);
        const float4 s4 = *reinterpret_cast<const float4 *>(bs + 4 * lane);      // code steps B_j / 127
        float rk[4] = {s4.x * (yk4.x * back_k), s4.y * (yk4.y * back_k), s4.z * (yk4.z * back_k), s4.w * (yk4.w * back_k)};
        float rq[4] = {s4.x * (yq4.x * back_q), s4.y * (yq4.y * back_q), s4.z * (yq4.z * back_q), s4.w * (yq4.w * back_q)};
        const float v4[4] = {__uint_as_float(v_raw.x << 16), __uint_as_float(v_raw.x & 0xFFFF0000u),
                             __uint_as_float(v_raw.y << 16), __uint_as_float(v_raw.y & 0xFFFF0000u)};
        LQ_TICK(6);
        named_arrive(bar0 + 2);                     // y has been read: the dot warp may put the record terms there
        named_wait(bar0 + 3);                       // the compensator projections are complete
        LQ_TICK(7);
#pragma unroll 2
        for (int h = 0; h < r; h++) {
          const uint2 w = *reinterpret_cast<const uint2 *>(cuh + h * D + 4 * lane);
          const float2 f01 = __half22float2(*reinterpret_cast<const __half2 *>(&w.x));
          const float2 f23 = __half22float2(*reinterpret_cast<const __half2 *>(&w.y));
          const float uc[4] = {f01.x, f01.y, f23.x, f23.y};
          const float pkh = pk[h], pqh = pq[h];
#pragma unroll
          for (int e = 0; e < 4; e++) { rk[e] = fmaf(uc[e], pkh, rk[e]); rq[e] = fmaf(uc[e], pqh, rq[e]); }
        }
        __syncwarp();                        // nobody reads the head block any more (the dot warp finished with
        {
          const int n_next = n_next_now();
          if (wanted(n_next)) request_head(bh_next, n_next);   // it before barrier 3): the next head's may land
        }
        named_wait(bar0 + 1);                       // the record terms are complete
        {
          const float4 tk = *reinterpret_cast<const float4 *>(y + 4 * lane);
          const float4 tq = *reinterpret_cast<const float4 *>(y + D + 4 * lane);
          rk[0] = rk[0] + tk.x; rk[1] = rk[1] + tk.y; rk[2] = rk[2] + tk.z; rk[3] = rk[3] + tk.w;
          rq[0] = rq[0] + tq.x; rq[1] = rq[1] + tq.y; rq[2] = rq[2] + tq.z; rq[3] = rq[3] + tq.w;
        }
        const float ktq = pq[r + (idx & 1)];
        float u[4], o[4];
#pragma unroll
        for (int e = 0; e < 4; e++) { u[e] = p.delta ? v4[e] - rk[e] : v4[e]; o[e] = fmaf(u[e], ktq, rq[e]); }
        LQ_TICK(8);
        *reinterpret_cast<float4 *>(p.o + bh * D + 4 * lane) = make_float4(o[0], o[1], o[2], o[3]);
        store4(p.record<rec_t>(bh, n, DIAG) + REC_U + 4 * lane, u[0], u[1], u[2], u[3]);
        if (FUSED && pass == 0) {
          __threadfence();
          named_arrive(bar0 + 5);
        }
      }
      LQ_TICK(9);
    }
  }
  if (FUSED && pass == 0 && role == 1 && lane == 0) {       // every head of this slot whose window fills has arrived
    __threadfence();
    atomicAdd(&g_fused_boundary_heads_done, 1u);
  }
#ifdef LQ_TIMING
  if (lane == 0)
    for (int i = 0; i < 12; i++) atomicAdd(&g_phase_cycles[16 * role + i], (unsigned long long)acc_[i]);
#endif
}

// Persistent kernel of two-warp CTAs: CTA `blockIdx.x` takes heads blockIdx.x, blockIdx.x + gridDim.x, ...
template <int GATE, bool R16, bool LONGW>
__global__ void __launch_bounds__(64, 6) decode_kernel(const Params p) {
  extern __shared__ __align__(128) unsigned char lq_slot[];
  LQ_STAMP(0, 0);
  // Resident while the kernel ahead drains: the CTA asks the L2 for its first head block meanwhile (a prefetch returns
  // no data, so it does not matter that the kernel ahead may still be writing that block: the L2 is where its writes
  // go).  The first head of a CTA is the only one whose copy nothing hides.
  if (threadIdx.x == 0 && blockIdx.x < static_cast<unsigned>(p.batch) * p.heads_v)
    bulk_prefetch_l2(p.head(blockIdx.x), head_bytes(p.r));
  const int lane = threadIdx.x & 31, role = threadIdx.x >> 5;
  uint32_t parA = 0, parR = 0;
  decode_slot_init<GATE, R16, false>(p, lq_slot, lane, role, 0, blockIdx.x, gridDim.x, nullptr);      // (shared memory only)
  grid_dependency_wait();                    // no data in global memory is read or written above this line
  LQ_STAMP(0, 1);
  decode_slot<GATE, R16, false, 0, LONGW>(p, lq_slot, lane, role, 0, blockIdx.x, gridDim.x, nullptr, parA, parR);
  LQ_STAMP(0, 3);
#ifdef LQ_TIMING
  if (threadIdx.x == 0 && blockIdx.x < 1024) {
    unsigned smid_;
    asm volatile("mov.u32 %0, %smid;" : "=r"(smid_));
    g_timeline[p.gen & 3][0][4][blockIdx.x] = smid_;
  }
  if (threadIdx.x == 32 && blockIdx.x < 1024) {          // the dot warp's last instruction
    unsigned long long t_;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));
    g_timeline[p.gen & 3][0][5][blockIdx.x] = t_;
  }
#endif
}

}  // namespace lq
