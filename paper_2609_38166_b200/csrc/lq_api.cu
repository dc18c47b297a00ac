// C boundary of the library: argument checks, launch configuration, and the kernels that wrap the
// device routines of lq_decode.cuh and lq_boundary.cuh.  Declarations and contracts: include/lq.h.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <map>
#include <mutex>
#include <tuple>

#include "lq_bf16w.cuh"
#include "lq_boundary.cuh"
#include "lq_decode.cuh"
#include "lq_fused.cuh"

namespace lq {

// ---------------------------------------------------------------------------------------------
// Boundary kernels: a CTA of 256 threads walks over heads (grid-stride) and takes those that need work.
// MODE 0: flush (window representation -> dense -> new window representation)
// MODE 1: quantize dense fp32 states         MODE 2: dequantize to dense fp32 states
// ---------------------------------------------------------------------------------------------
// RM: the largest r the instance handles (4, 8 or MAX_R; the fit keeps its small matrices in registers, RM wide).
template <int GATE, int MODE, bool R16, int RM>
__global__ void __launch_bounds__(256, 2) boundary_kernel(const Params p, const int stage_bufs) {
  extern __shared__ float4 lq_smem4[];
  float *smem = reinterpret_cast<float *>(lq_smem4);
  constexpr bool DIAG = GATE == LQ_GATE_DIAG;
  const Tile t;
  const size_t nh = (size_t)p.batch * p.heads_v;
  __shared__ uint32_t todo_mask;
  __shared__ int todo_n[32];
  LQ_STAMP(1, 0);
#ifdef LQ_TIMING
  if (threadIdx.x == 0 && blockIdx.x < 1024) {
    unsigned smid_;
    asm volatile("mov.u32 %0, %smid;" : "=r"(smid_));
    g_timeline[p.gen & 3][1][5][blockIdx.x] = smid_;
  }
#endif
  grid_dependency_wait();                    // everything the kernel before this one wrote is visible from here on
  LQ_STAMP(1, 1);
  // the decode kernel ahead of a flush counts the tickets of its pool of heads in the state's scratch words
  if (MODE == 0 && p.work != nullptr && blockIdx.x == 0 && threadIdx.x == 0) p.work[0] = 0;
#ifdef LQ_TIMING
  if (threadIdx.x == 0) { for (int i = 0; i < 16; i++) lq_bacc[i] = 0; lq_btick = clock64(); }
  bool first_flush_ = true;
#endif
  // The CTA owns heads blockIdx.x + k * gridDim.x.  Warp 0 looks at 32 of them at a time (one load each, all in
  // flight together) and publishes which ones have work and how many records each holds; then the CTA takes
  // them one after the other, fetching the next one's data into the other staging buffer meanwhile.
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
      // The arrival on win_pos (arrive_and_set: the last head of a sequence to arrive stores 0) only says "this head
      // has read the old value", which it just did; nobody inside this kernel waits for the 0.  Made here, 32 heads
      // at once, the atomic's round trip hides behind the wait for the first staging buffer.
      if (MODE == 0 && want) arrive_and_set(p.win_pos, static_cast<int>(cand / p.heads_v), p.heads_v, 0);
    }
    __syncthreads();
    LQ_BTICK(0);
    uint32_t mask = todo_mask;
    int buf = 0;
    bool staged = false;                     // the data of the head about to be processed is already on its way
    while (mask) {
      const int kbit = __ffs(mask) - 1;
      mask &= mask - 1;
      const size_t bh = base + kbit * (size_t)gridDim.x;
      const int b = static_cast<int>(bh / p.heads_v);
      const int n = todo_n[kbit];
      const BoundarySmem sm(smem, p.W, p.r, DIAG, R16, buf);
      float M[8][8];
      if (MODE == 1) {
        const float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
        for (int a = 0; a < 8; a++) load8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);
      } else {
        // (the barrier that ended the previous head's work also freed both staging buffers for writing)
        if (!staged) {
          stage_issue<GATE, R16>(p, sm, t, bh, n);
          cp_async_commit();
        }
        staged = false;
        if (mask && stage_bufs > 1) {
          const int knext = __ffs(mask) - 1;
          const BoundarySmem nx(smem, p.W, p.r, DIAG, R16, buf ^ 1);
          stage_issue<GATE, R16>(p, nx, t, base + knext * (size_t)gridDim.x, todo_n[knext]);
          cp_async_commit();
          staged = true;
          cp_async_wait_but_one();
        } else {
          cp_async_wait_all();
        }
        __syncthreads();
        LQ_BTICK(1);
#ifdef LQ_TIMING
        if (first_flush_) LQ_STAMP(1, 2);
#endif
        reconstruct_tile<GATE, R16>(p, sm, t, bh, n, M);
      }
      if (MODE == 2) {
        float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
        for (int a = 0; a < 8; a++) store8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);
      } else {
        quantize_tile<RM>(p, sm, t, bh, MODE == 0 ? n : 0, M);
      }
      __syncthreads();                       // this head's use of shared memory is over
      LQ_BTICK(9);
#ifdef LQ_TIMING
      if (first_flush_) LQ_STAMP(1, 3);
      first_flush_ = false;
#endif
      if (MODE == 1 && t.tid == 0) p.win_pos[b] = 0;      // (nobody reads win_pos in this mode)
      if (staged) buf ^= 1;
    }
    __syncthreads();                         // todo_mask / todo_n are rewritten by the next round
  }
#ifdef LQ_TIMING
  LQ_STAMP(1, 4);
  if (threadIdx.x == 0) {
    for (int i = 0; i < 16; i++) atomicAdd(&g_phase_cycles[32 + i], (unsigned long long)lq_bacc[i]);
  }
#endif
}

// ---------------------------------------------------------------------------------------------
// Baseline: Eq. 1 on a dense state that is read and written in full every token.
// ---------------------------------------------------------------------------------------------
template <int GATE, bool BF16>
__global__ void __launch_bounds__(256, (BF16 || GATE == LQ_GATE_SCALAR) ? 3 : 2) ref_kernel(const Params p) {
  __shared__ __align__(16) float kt_s[D], q_s[D], bv_s[D], a_s[D], col_s[D], part_s[8 * D];
  const Tile t;
  const size_t bh = blockIdx.x;
  const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);
  float M[8][8];
  if (BF16) {
    const uint16_t *S = p.S16 + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) {
      const uint4 w = __ldcs(reinterpret_cast<const uint4 *>(S + (8 * t.ty + a) * D + 8 * t.tx));   // streamed: read once
      const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; e++) {
        M[a][2 * e] = __uint_as_float(ws[e] << 16);
        M[a][2 * e + 1] = __uint_as_float(ws[e] & 0xFFFF0000u);
      }
    }
  } else {
    const float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) load8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);   // (streaming hints slow this one down)
  }
  if (t.tid < D) {
    const int group = p.heads_v / p.heads_qk;
    const size_t qk_off = ((size_t)b * p.heads_qk + hv / group) * D;
    const float k_i = bf16_bits(p.k[qk_off + t.tid]);
    const float a_i = GATE == LQ_GATE_DIAG ? bf16_bits(p.alpha[bh * D + t.tid]) : bf16_bits(p.alpha[bh]);
    kt_s[t.tid] = bf16_bits(p.beta[bh]) * k_i;
    bv_s[t.tid] = a_i * k_i;
    a_s[t.tid] = a_i;
    q_s[t.tid] = bf16_bits(p.q[qk_off + t.tid]);
  }
  __syncthreads();
  float x[8], pc[8], u[8], o[8], kt[8], ai[8];
  load8(bv_s + 8 * t.ty, x);
  col_blocks(M, x, pc);
  col_tree(pc, part_s, col_s, t, u);                           // S^T (alpha.k)
#pragma unroll
  for (int c = 0; c < 8; c++) {                               // b = 0 (no delta rule): nothing is subtracted
    const float vc = bf16_bits(p.v[bh * D + 8 * t.tx + c]);
    u[c] = p.delta ? vc - u[c] : vc;
  }
  load8(kt_s + 8 * t.ty, kt);
  load8(a_s + 8 * t.ty, ai);
#pragma unroll
  for (int a = 0; a < 8; a++)
#pragma unroll
    for (int c = 0; c < 8; c++) M[a][c] = fmaf(kt[a], u[c], ai[a] * M[a][c]);
  load8(q_s + 8 * t.ty, x);
  col_blocks(M, x, pc);
  col_tree(pc, part_s, col_s, t, o);
  if (t.ty == 0) store8(p.o + bh * D + 8 * t.tx, o);
  if (BF16) {
    uint16_t *S = p.S16 + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) {
      uint32_t ws[4];
#pragma unroll
      for (int e = 0; e < 4; e++)
        ws[e] = (uint32_t)to_bf16_bits(M[a][2 * e]) | ((uint32_t)to_bf16_bits(M[a][2 * e + 1]) << 16);
      __stcs(reinterpret_cast<uint4 *>(S + (8 * t.ty + a) * D + 8 * t.tx), make_uint4(ws[0], ws[1], ws[2], ws[3]));
    }
  } else {
    float *S = p.S + bh * (size_t)(D * D);
#pragma unroll
    for (int a = 0; a < 8; a++) store8(S + (8 * t.ty + a) * D + 8 * t.tx, M[a]);
  }
}

// ---------------------------------------------------------------------------------------------
// The window representation as separate arrays in the paper's orientation <-> the packed layout of lq_state
// (lq_import_state / lq_export_state): pure data movement, one CTA per head.
// ---------------------------------------------------------------------------------------------
template <bool IMPORT>
__global__ void __launch_bounds__(256) convert_state_kernel(const Params p, const lq_state_arrays a, const int diag) {
  __shared__ __align__(16) int8_t tile[D][D + 16];            // the code matrix on its way through the transposition
  const size_t bh = blockIdx.x;
  const int tid = threadIdx.x, W = p.W, r = p.r;
  const int b = static_cast<int>(bh / p.heads_v), hv = static_cast<int>(bh % p.heads_v);
  int8_t *Z = a.codes + bh * (size_t)(D * D);                 // [d_k][d_v]
  int8_t *ZT = p.codes(bh);                                   // [d_v][d_k]
  const int8_t *src = IMPORT ? Z : ZT;
  int8_t *dst = IMPORT ? ZT : Z;
  for (int e = tid; e < D * D / 16; e += 256) {
    const int row = e >> 3, c16 = e & 7;
    *reinterpret_cast<uint4 *>(&tile[row][16 * c16]) = *reinterpret_cast<const uint4 *>(src + row * D + 16 * c16);
  }
  __syncthreads();
  for (int e = tid; e < D * D / 16; e += 256) {
    const int row = e >> 3, c16 = e & 7;
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; q++) {
      uint32_t x = 0;
#pragma unroll
      for (int j = 0; j < 4; j++) x |= static_cast<uint32_t>(static_cast<uint8_t>(tile[16 * c16 + 4 * q + j][row])) << (8 * j);
      w[q] = x;
    }
    *reinterpret_cast<uint4 *>(dst + row * D + 16 * c16) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  auto move = [&](auto *packed, auto *plain) {
    if (IMPORT) *packed = *plain;
    else *plain = *packed;
  };
  if (tid < D) {
    move(p.col_scale(bh) + tid, a.col_scale + bh * D + tid);
    move(p.row_smooth(bh) + tid, a.row_smooth + bh * D + tid);
  }
  for (int e = tid; e < r * D; e += 256) {
    move(p.comp_k(bh) + e, a.comp_k + bh * (size_t)(r * D) + e);
    move(p.comp_u(bh) + e, a.comp_u + bh * (size_t)(r * D) + e);
  }
  const int RF = record_floats(diag != 0);
  auto move_record = [&](int j, int off, float *plain) {       // one element of record j, fp32 or fp16 in the packed rows
    if (p.rec16) {
      __half *row = p.record<__half>(bh, j, diag != 0);
      if (IMPORT) row[off] = __ushort_as_half(to_f16_bits_sat(*plain));
      else *plain = __half2float(row[off]);
    } else {
      float *row = p.record<float>(bh, j, diag != 0);
      if (IMPORT) row[off] = *plain;
      else *plain = row[off];
    }
  };
  for (int e = tid; e < W * D; e += 256) {
    const int j = e / D, i = e % D;
    move_record(j, REC_KT + i, a.buf_k + (bh * W + j) * (size_t)D + i);
    move_record(j, REC_U + i, a.buf_u + (bh * W + j) * (size_t)D + i);
    if (diag) move_record(j, REC_A + i, a.buf_a + (bh * W + j) * (size_t)D + i);
  }
  if (!diag && tid < W) move(p.decays + bh * (size_t)W + tid, a.buf_a + bh * (size_t)W + tid);
  if (hv == 0 && tid == 0) move(p.win_pos + b, a.win_pos + b);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

static lq_status check_shape(const lq_shape *s) {
  if (!s) return LQ_ERR_NULL;
  if (s->batch < 0 || s->heads_v <= 0 || s->heads_qk <= 0 || s->d_k <= 0 || s->d_v <= 0 || s->W <= 0 || s->r < 0 ||
      s->n_iter < 1 || s->heads_v % s->heads_qk != 0 || (s->gate != LQ_GATE_SCALAR && s->gate != LQ_GATE_DIAG) ||
      (s->delta != 0 && s->delta != 1) || (s->rec16 != 0 && s->rec16 != 1) ||
      (s->state_bf16 != 0 && s->state_bf16 != 1) || (s->state_bf16 && (s->r != 0 || s->smooth != 0)))
    return LQ_ERR_SHAPE;
  if (s->d_k != D || s->d_v != D || s->W > MAX_W || s->r > MAX_R) return LQ_ERR_UNSUPPORTED;
  return LQ_OK;
}

static lq_status check_ptrs(std::initializer_list<const void *> ptrs) {
  for (const void *q : ptrs)
    if (!q) return LQ_ERR_NULL;
  for (const void *q : ptrs)
    if (!aligned16(q)) return LQ_ERR_ALIGN;
  return LQ_OK;
}

// arrays that are only read or written one element at a time need their natural alignment only
static lq_status check_scalar_ptrs(std::initializer_list<const void *> ptrs, unsigned elem_bytes) {
  for (const void *q : ptrs)
    if (!q) return LQ_ERR_NULL;
  for (const void *q : ptrs)
    if (reinterpret_cast<uintptr_t>(q) & (elem_bytes - 1)) return LQ_ERR_ALIGN;
  return LQ_OK;
}

static lq_status check_state(const lq_shape *s, const lq_state *st, bool need_buffers) {
  if (!st) return LQ_ERR_NULL;
  lq_status rc = check_ptrs({st->heads});
  if (rc != LQ_OK) return rc;
  if ((rc = check_scalar_ptrs({st->win_pos}, 4)) != LQ_OK) return rc;
  if (st->work && (reinterpret_cast<uintptr_t>(st->work) & 3u)) return LQ_ERR_ALIGN;
  if (need_buffers) {
    if ((rc = check_ptrs({st->records})) != LQ_OK) return rc;
    if (s->gate == LQ_GATE_SCALAR && (rc = check_scalar_ptrs({st->decays}, 4)) != LQ_OK) return rc;
  }
  return LQ_OK;
}

static Params make_params(const lq_shape *s, const lq_state *st) {
  Params p{};
  p.batch = s->batch; p.heads_v = s->heads_v; p.heads_qk = s->heads_qk; p.W = s->W; p.r = s->r;
  p.n_iter = s->n_iter; p.smooth = s->smooth; p.delta = s->delta; p.rec16 = s->rec16; p.force = 0;
  if (st) {
    p.heads = st->heads; p.records = st->records; p.decays = st->decays; p.win_pos = st->win_pos;
    p.work = st->work;
  }
  return p;
}

static int sm_count() {
  static int cached = 0;
  if (!cached) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
      cached = n;
    else
      return 148;
  }
  return cached;
}

// What a launch needs to ask the runtime only once per (device, kernel): the opt-in to more than 48 KB of shared
// memory and the number of CTAs of a kernel that an SM holds.  Both calls cost a few microseconds of host time,
// which a step of two to ten launches would otherwise pay every token.
static int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return dev;
}

// (the opt-in is needed once static + dynamic shared memory pass 48 KB; the kernels here hold up to 20 KB static)
static bool smem_opt_in(const void *kernel, size_t smem) {
  if (smem <= 24 * 1024) return true;
  static std::mutex m;
  static std::map<std::pair<int, const void *>, size_t> granted;
  std::lock_guard<std::mutex> lock(m);
  size_t &have = granted[{current_device(), kernel}];
  if (have >= smem) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  have = smem;
  return true;
}

// resident CTAs per SM of `kernel` with this block size and dynamic shared memory (0: the query failed)
static int ctas_per_sm(const void *kernel, int block, size_t smem) {
  static std::mutex m;
  static std::map<std::tuple<int, const void *, int, size_t>, int> known;
  std::lock_guard<std::mutex> lock(m);
  int &per_sm = known[std::make_tuple(current_device(), kernel, block, smem)];
  if (per_sm > 0) return per_sm;
  int v = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, kernel, block, smem) != cudaSuccess || v < 1) {
    cudaGetLastError();
    return 0;
  }
  return per_sm = v;
}

template <typename K, typename P>
static lq_status launch(K kernel, int grid, int block, size_t smem, cudaStream_t stream, const P &p) {
  if (grid <= 0) return LQ_OK;
  if (!smem_opt_in(reinterpret_cast<const void *>(kernel), smem)) return LQ_ERR_CUDA;
  kernel<<<grid, block, smem, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}

// Launch that may begin while the kernel before it on the stream is still draining (programmatic dependent
// launch): its CTAs become resident as SM resources free up and sit in griddepcontrol.wait until that kernel
// has completed and its writes are visible.  Only for kernels that execute griddepcontrol.wait before their
// first access to global memory.
template <typename K, typename... Args>
static lq_status launch_dependent(K kernel, int grid, int block, size_t smem, cudaStream_t stream, const Args &...args) {
  if (grid <= 0) return LQ_OK;
  if (!smem_opt_in(reinterpret_cast<const void *>(kernel), smem)) return LQ_ERR_CUDA;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, args...) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  return LQ_OK;
}

// grid <= min(work items, CTAs that fit on the device at once), for kernels that stride over their work
template <typename K>
static lq_status launch_persistent(K kernel, long items, int block, size_t smem, cudaStream_t stream, const Params &p) {
  if (items <= 0) return LQ_OK;
  if (!smem_opt_in(reinterpret_cast<const void *>(kernel), smem)) return LQ_ERR_CUDA;
  const int per_sm = ctas_per_sm(reinterpret_cast<const void *>(kernel), block, smem);
  if (per_sm < 1) return LQ_ERR_CUDA;
  const long resident = (long)per_sm * sm_count();
  // Every CTA takes ceil(items / resident) items at most; the smallest grid with that property leaves no last
  // round in which a fraction of the CTAs works while the others have left (8192 heads: 820 CTAs of 10 heads
  // instead of 888 of which 200 take a tenth).  With scratch words in the state the items of a partial last round
  // go to the CTAs that get there first (decode_slot), and every CTA that fits is launched.
  const long rounds = (items + resident - 1) / resident;
  const long grid = p.work != nullptr ? (items < resident ? items : resident) : (items + rounds - 1) / rounds;
  return launch_dependent(kernel, static_cast<int>(grid), block, smem, stream, p);
}

// per-window BF16: persistent CTAs that stride over the heads
template <int MODE>
static lq_status launch_bf16w_boundary(const lq_shape *s, const Params &p, cudaStream_t stream) {
  const bool diag = s->gate == LQ_GATE_DIAG;
  const bool r16 = MODE != 1 && s->rec16 != 0;
  const size_t smem = bf16w_boundary_smem(s->W, diag, r16);
  const long nh = (long)s->batch * s->heads_v;
  const int grid = static_cast<int>(nh < 2L * sm_count() ? nh : 2L * sm_count());      // persistent, two per SM
  if (r16)
    return diag ? launch_dependent(bf16w_boundary_kernel<LQ_GATE_DIAG, MODE == 1 ? 0 : MODE, true>, grid, 256, smem, stream, p)
                : launch_dependent(bf16w_boundary_kernel<LQ_GATE_SCALAR, MODE == 1 ? 0 : MODE, true>, grid, 256, smem, stream, p);
  return diag ? launch_dependent(bf16w_boundary_kernel<LQ_GATE_DIAG, MODE, false>, grid, 256, smem, stream, p)
              : launch_dependent(bf16w_boundary_kernel<LQ_GATE_SCALAR, MODE, false>, grid, 256, smem, stream, p);
}

template <int MODE>
static lq_status launch_boundary(const lq_shape *s, const Params &p, cudaStream_t stream) {
  if (s->state_bf16) return launch_bf16w_boundary<MODE>(s, p, stream);
  const bool diag = s->gate == LQ_GATE_DIAG;
  const bool r16 = MODE != 1 && s->rec16 != 0;               // quantizing a dense state reads no records
  const int bufs = MODE == 1 ? 1 : BoundarySmem::buffers(s->W, s->r, diag, r16);
  const size_t smem = BoundarySmem::bytes(s->W, s->r, diag, r16, bufs);
  const long nh = (long)s->batch * s->heads_v;
  // persistent: the CTAs that are resident at once (two per SM), each striding over the heads
  const int grid = static_cast<int>(nh < 2L * sm_count() ? nh : 2L * sm_count());
  // the flush (the hot one) is compiled for r <= 4, r <= 8 and any r; the others once
  constexpr int M_ = MODE;
  if (MODE == 0 && s->r <= 4) {
    if (r16) return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, M_, true, 4>, grid, 256, smem, stream, p, bufs)
                         : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, M_, true, 4>, grid, 256, smem, stream, p, bufs);
    return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, M_, false, 4>, grid, 256, smem, stream, p, bufs)
                : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, M_, false, 4>, grid, 256, smem, stream, p, bufs);
  }
  if (MODE == 0 && s->r <= 8) {
    if (r16) return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, M_, true, 8>, grid, 256, smem, stream, p, bufs)
                         : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, M_, true, 8>, grid, 256, smem, stream, p, bufs);
    return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, M_, false, 8>, grid, 256, smem, stream, p, bufs)
                : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, M_, false, 8>, grid, 256, smem, stream, p, bufs);
  }
  if (r16)
    return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, MODE == 1 ? 0 : MODE, true, MAX_R>, grid, 256, smem, stream, p, bufs)
                : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, MODE == 1 ? 0 : MODE, true, MAX_R>, grid, 256, smem, stream, p, bufs);
  return diag ? launch_dependent(boundary_kernel<LQ_GATE_DIAG, MODE, false, MAX_R>, grid, 256, smem, stream, p, bufs)
              : launch_dependent(boundary_kernel<LQ_GATE_SCALAR, MODE, false, MAX_R>, grid, 256, smem, stream, p, bufs);
}

// The step as one cooperative kernel (lq_fused.cuh): one decode CTA and one boundary CTA per SM.
static bool fused_step_wanted(long nh) {
  // Off unless LQ_FUSED_STEP=1 is set: on B200 the fused kernel is slower than the two kernels (a boundary CTA
  // alone on an SM is latency-bound and takes 21 us per head where two of them sharing an SM take 12 us each,
  // and the registers of an SM do not hold two boundary CTAs next to the decode slots).
  (void)nh;
  const char *e = getenv("LQ_FUSED_STEP");
  return e && atoi(e) != 0;
}

template <int GATE, bool R16>
static lq_status launch_fused_step_t(const lq_shape *s, const Params &p, cudaStream_t stream) {
  const bool diag = GATE == LQ_GATE_DIAG;
  const size_t smem = fused_smem_bytes(s->W, s->r, diag, R16);
  auto kernel = fused_step_kernel<GATE, R16>;
  if (smem > 227 * 1024) return LQ_ERR_UNSUPPORTED;
  if (!smem_opt_in(reinterpret_cast<const void *>(kernel), smem)) return LQ_ERR_UNSUPPORTED;
  if (ctas_per_sm(reinterpret_cast<const void *>(kernel), 256, smem) < 2)
    return LQ_ERR_UNSUPPORTED;               // two CTAs per SM are the design
  const long nh = (long)s->batch * s->heads_v;
  const int sms = sm_count();
  if (nh > (long)sms * FUSED_SLOTS * FUSED_NBUF || nh > (long)sms * 2048) return LQ_ERR_UNSUPPORTED;
  int decode_ctas = sms;
  Params pp = p;
  void *args[] = {&pp, &decode_ctas};
  if (cudaLaunchCooperativeKernel(reinterpret_cast<void *>(kernel), dim3(2 * sms), dim3(256), args, smem, stream) !=
      cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  return LQ_OK;
}

static lq_status launch_fused_step(const lq_shape *s, const Params &p, cudaStream_t stream) {
  const bool diag = s->gate == LQ_GATE_DIAG;
  if (s->rec16) return diag ? launch_fused_step_t<LQ_GATE_DIAG, true>(s, p, stream) : launch_fused_step_t<LQ_GATE_SCALAR, true>(s, p, stream);
  return diag ? launch_fused_step_t<LQ_GATE_DIAG, false>(s, p, stream) : launch_fused_step_t<LQ_GATE_SCALAR, false>(s, p, stream);
}

}  // namespace lq

using namespace lq;

extern "C" {

static lq_status decode_step_impl(const lq_shape *shape, const lq_state *state, const uint16_t *q, const uint16_t *k,
                                  const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                  lq_stream stream, cudaEvent_t between) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;
  if ((rc = check_ptrs({q, k, v, o})) != LQ_OK) return rc;
  if ((rc = check_scalar_ptrs({beta}, 2)) != LQ_OK) return rc;
  if ((rc = shape->gate == LQ_GATE_DIAG ? check_ptrs({alpha}) : check_scalar_ptrs({alpha}, 2)) != LQ_OK) return rc;
  Params p = make_params(shape, state);
#ifdef LQ_TIMING
  static int generation = 0;
  p.gen = generation++;
#endif
  p.q = q; p.k = k; p.v = v; p.beta = beta; p.alpha = alpha; p.o = o;
  const bool diag = shape->gate == LQ_GATE_DIAG;
  const long nh = (long)shape->batch * shape->heads_v;
  // persistent two-warp CTAs, each with its own shared-memory slot: as many as are resident at once
  const bool r16 = shape->rec16 != 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (shape->state_bf16) {                   // per-window BF16: one CTA per head
    const int grid = static_cast<int>(nh);
    const size_t rsm = bf16w_decode_smem(shape->W, diag, r16);
    if (r16)
      rc = diag ? launch_dependent(bf16w_decode_kernel<LQ_GATE_DIAG, true>, grid, 256, rsm, st, p)
                : launch_dependent(bf16w_decode_kernel<LQ_GATE_SCALAR, true>, grid, 256, rsm, st, p);
    else
      rc = diag ? launch_dependent(bf16w_decode_kernel<LQ_GATE_DIAG, false>, grid, 256, rsm, st, p)
                : launch_dependent(bf16w_decode_kernel<LQ_GATE_SCALAR, false>, grid, 256, rsm, st, p);
    if (rc != LQ_OK) return rc;
    if (between && cudaEventRecord(between, st) != cudaSuccess) {
      cudaGetLastError();
      return LQ_ERR_CUDA;
    }
    return launch_boundary<0>(shape, p, st);
  }
  if (!between && fused_step_wanted(nh)) {
    lq_status frc = launch_fused_step(shape, p, st);
    if (frc != LQ_ERR_UNSUPPORTED) return frc;       // does not fit this device or shape: the two kernels below
  }
  const size_t smem = DecodeSlot(shape->W, shape->r, diag, r16).bytes;
  const bool longw = shape->W - 1 > REC_SEG;               // windows whose records come in more than one segment
  if (longw) {
    if (r16)
      rc = diag ? launch_persistent(decode_kernel<LQ_GATE_DIAG, true, true>, nh, 64, smem, st, p)
                : launch_persistent(decode_kernel<LQ_GATE_SCALAR, true, true>, nh, 64, smem, st, p);
    else
      rc = diag ? launch_persistent(decode_kernel<LQ_GATE_DIAG, false, true>, nh, 64, smem, st, p)
                : launch_persistent(decode_kernel<LQ_GATE_SCALAR, false, true>, nh, 64, smem, st, p);
  } else {
    if (r16)
      rc = diag ? launch_persistent(decode_kernel<LQ_GATE_DIAG, true, false>, nh, 64, smem, st, p)
                : launch_persistent(decode_kernel<LQ_GATE_SCALAR, true, false>, nh, 64, smem, st, p);
    else
      rc = diag ? launch_persistent(decode_kernel<LQ_GATE_DIAG, false, false>, nh, 64, smem, st, p)
                : launch_persistent(decode_kernel<LQ_GATE_SCALAR, false, false>, nh, 64, smem, st, p);
  }
  if (rc != LQ_OK) return rc;
  if (between && cudaEventRecord(between, st) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  return launch_boundary<0>(shape, p, st);     // sequences whose window just became full
}

lq_status lq_decode_step(const lq_shape *shape, const lq_state *state, const uint16_t *q, const uint16_t *k,
                         const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o, lq_stream stream) {
  return decode_step_impl(shape, state, q, k, v, beta, alpha, o, stream, nullptr);
}

lq_status lq_decode_step_profiled(const lq_shape *shape, const lq_state *state, const uint16_t *q, const uint16_t *k,
                                  const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                  lq_stream stream, void *event_between) {
  return decode_step_impl(shape, state, q, k, v, beta, alpha, o, stream, static_cast<cudaEvent_t>(event_between));
}

uint64_t lq_head_bytes(const lq_shape *s) {
  if (check_shape(s) != LQ_OK) return 0;
  return s->state_bf16 ? (uint64_t)BF16W_HEAD_BYTES : (uint64_t)head_bytes(s->r);
}

uint64_t lq_record_floats(const lq_shape *s) {
  return check_shape(s) == LQ_OK ? (uint64_t)record_floats(s->gate == LQ_GATE_DIAG) : 0;
}

uint64_t lq_decode_stage_bytes(const lq_shape *s) {
  if (check_shape(s) != LQ_OK) return 0;
  const uint64_t B = s->batch, Hv = s->heads_v, Hqk = s->heads_qk, K = s->d_k, V = s->d_v;
  auto up = [](uint64_t x) { return (x + 255) / 256 * 256; };
  const uint64_t na = s->gate == LQ_GATE_DIAG ? B * Hv * K : B * Hv;
  return 2 * up(2 * B * Hqk * K) + up(2 * B * Hv * V) + up(2 * B * Hv) + up(2 * na) + up(4 * B * Hv * V);
}

}  // extern "C"

// One launch that brings the five input arrays from mapped pinned host memory into the device staging
// buffer (the alternative, five cudaMemcpyAsync calls, costs about 10 us of latency per copy on top of the
// transfer itself).  Every segment is a whole number of 16-byte units; both ends are 16-byte aligned.
namespace {
struct GatherSegs {
  const uint4 *src[5];
  uint4 *dst[5];
  uint32_t units[5];      // 16-byte units per segment
};
__global__ void __launch_bounds__(256) gather_kernel(const GatherSegs g) {
  const uint32_t stride = gridDim.x * blockDim.x;
#pragma unroll
  for (int sgm = 0; sgm < 5; sgm++) {
    const uint4 *__restrict__ src = g.src[sgm];
    uint4 *__restrict__ dst = g.dst[sgm];
    const uint32_t n = g.units[sgm];
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n; i += 4 * stride) {          // four loads in flight per thread
      const uint4 a = src[i], b = src[i + stride], c = src[i + 2 * stride], d = src[i + 3 * stride];
      dst[i] = a; dst[i + stride] = b; dst[i + 2 * stride] = c; dst[i + 3 * stride] = d;
    }
    for (; i < n; i += stride) dst[i] = src[i];
  }
}

// The device alias of a pinned, mapped host pointer; null if the memory is not mapped into the device.
template <typename T>
T *device_alias(T *host) {
  void *dev = nullptr;
  if (cudaHostGetDevicePointer(&dev, const_cast<void *>(static_cast<const void *>(host)), 0) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return static_cast<T *>(dev);
}
}  // namespace

extern "C" {

static void host_pipe_break_chain();

static lq_status host_step_impl(const lq_shape *shape, const lq_state *state, const uint16_t *q_h, const uint16_t *k_h,
                                const uint16_t *v_h, const uint16_t *beta_h, const uint16_t *alpha_h, float *o_h,
                                void *stage, lq_stream stream, bool direct_ok) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;     // nothing is enqueued before every argument is checked
  if (!q_h || !k_h || !v_h || !beta_h || !alpha_h || !o_h || !stage) return LQ_ERR_NULL;
  if (!aligned16(stage)) return LQ_ERR_ALIGN;
  const uint64_t B = shape->batch, Hv = shape->heads_v, Hqk = shape->heads_qk, K = shape->d_k, V = shape->d_v;
  auto up = [](uint64_t x) { return (x + 255) / 256 * 256; };
  const uint64_t nqk = 2 * B * Hqk * K, nv = 2 * B * Hv * V, nb = 2 * B * Hv;
  const uint64_t na = 2 * (shape->gate == LQ_GATE_DIAG ? B * Hv * K : B * Hv), no = 4 * B * Hv * V;
  char *base = static_cast<char *>(stage);
  uint16_t *q_d = reinterpret_cast<uint16_t *>(base); base += up(nqk);
  uint16_t *k_d = reinterpret_cast<uint16_t *>(base); base += up(nqk);
  uint16_t *v_d = reinterpret_cast<uint16_t *>(base); base += up(nv);
  uint16_t *b_d = reinterpret_cast<uint16_t *>(base); base += up(nb);
  uint16_t *a_d = reinterpret_cast<uint16_t *>(base); base += up(na);
  float *o_d = reinterpret_cast<float *>(base);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (B == 0) return LQ_OK;
  host_pipe_break_chain();                   // this call writes `stage` in stream order only

  // Fast path, when all six host arrays are pinned, mapped into the device and 16-byte aligned: one gather
  // launch reads the inputs over the bus, and the decode kernel writes o straight into the host array (posted
  // writes that overlap the kernel), so no copy follows the step.
  const uint16_t *src_h[5] = {q_h, k_h, v_h, beta_h, alpha_h};
  uint16_t *dst_d[5] = {q_d, k_d, v_d, b_d, a_d};
  const uint64_t bytes[5] = {nqk, nqk, nv, nb, na};
  GatherSegs g;
  bool mapped = direct_ok && aligned16(o_h) && no < (1ull << 35);
  for (int i = 0; mapped && i < 5; i++) {
    const uint16_t *alias = (aligned16(src_h[i]) && bytes[i] < (1ull << 35)) ? device_alias(src_h[i]) : nullptr;
    mapped = alias != nullptr;
    g.src[i] = reinterpret_cast<const uint4 *>(alias);
    g.dst[i] = reinterpret_cast<uint4 *>(dst_d[i]);
    g.units[i] = static_cast<uint32_t>((bytes[i] + 15) / 16);   // the regions of `stage` are padded to 256 bytes;
  }                                                             // a ragged tail is covered below
  float *o_alias = mapped ? device_alias(o_h) : nullptr;
  // a segment that is not a whole number of 16-byte units would read past the end of the host array
  for (int i = 0; mapped && i < 5; i++) mapped = bytes[i] % 16 == 0;
  if (mapped && o_alias) {
    rc = launch(gather_kernel, 2 * sm_count(), 256, 0, st, g);
    if (rc != LQ_OK) return rc;
    return lq_decode_step(shape, state, q_d, k_d, v_d, b_d, a_d, o_alias, stream);
  }

  if (cudaMemcpyAsync(q_d, q_h, nqk, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(k_d, k_h, nqk, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(v_d, v_h, nv, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(b_d, beta_h, nb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(a_d, alpha_h, na, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  rc = lq_decode_step(shape, state, q_d, k_d, v_d, b_d, a_d, o_d, stream);
  if (rc != LQ_OK) return rc;
  if (cudaMemcpyAsync(o_h, o_d, no, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  return LQ_OK;
}

lq_status lq_decode_step_host(const lq_shape *shape, const lq_state *state, const uint16_t *q_h, const uint16_t *k_h,
                              const uint16_t *v_h, const uint16_t *beta_h, const uint16_t *alpha_h, float *o_h,
                              void *stage, lq_stream stream) {
  return host_step_impl(shape, state, q_h, k_h, v_h, beta_h, alpha_h, o_h, stage, stream, true);
}

// ---------------------------------------------------------------------------------------------
// Host-buffer decode step with the copies overlapped with the kernels: the batch is cut into chunks of
// sequences; chunk c+1 is copied in and chunk c-1 copied out while chunk c is computed.  The copies run on two
// streams that the library creates per device on first use; events tie them to the caller's stream, so for the
// caller the call is still one piece of work on `stream`.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int PIPE_CHUNKS = 2;
struct HostPipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t start = nullptr, out = nullptr, in[PIPE_CHUNKS] = {}, done[PIPE_CHUNKS] = {};
  // The previous pipelined call on this device, if the next one may chain onto it: same staging buffer, stream
  // and staging layout.  done[c] then still marks the moment that call's decode kernel had consumed the inputs
  // of sub-batch c.
  bool chain = false;
  const void *stage = nullptr;
  cudaStream_t stream = nullptr;
  uint64_t layout[5] = {};                   // B, Hv, Hqk, gate, W
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];

lq_status host_pipe(HostPipe **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  HostPipe &hp = g_pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.out, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; ok && c < PIPE_CHUNKS; c++)
      ok = cudaEventCreateWithFlags(&hp.in[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return LQ_ERR_CUDA;
    }
    hp.ready = true;
  }
  *out = &hp;
  return LQ_OK;
}
}  // namespace

// a later pipelined call must not start reading its inputs early: something else is about to use a staging buffer
static void host_pipe_break_chain() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return;
  }
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  g_pipes[dev].chain = false;
}

lq_status lq_decode_step_host_pipelined(const lq_shape *shape, const lq_state *state, const uint16_t *q_h,
                                        const uint16_t *k_h, const uint16_t *v_h, const uint16_t *beta_h,
                                        const uint16_t *alpha_h, float *o_h, void *stage, lq_stream stream) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if (shape->batch < 8 * PIPE_CHUNKS)          // nothing to overlap (breaks a chain of pipelined calls as well)
    return lq_decode_step_host(shape, state, q_h, k_h, v_h, beta_h, alpha_h, o_h, stage, stream);
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;
  if (!q_h || !k_h || !v_h || !beta_h || !alpha_h || !o_h || !stage) return LQ_ERR_NULL;
  if (!aligned16(stage)) return LQ_ERR_ALIGN;
  const uint64_t B = shape->batch, Hv = shape->heads_v, Hqk = shape->heads_qk, K = shape->d_k, V = shape->d_v;
  const bool diag = shape->gate == LQ_GATE_DIAG;
  auto up = [](uint64_t x) { return (x + 255) / 256 * 256; };
  const uint64_t eqk = Hqk * K, ev = Hv * V, eb = Hv, ea = diag ? Hv * K : Hv;   // elements per sequence
  char *base = static_cast<char *>(stage);
  uint16_t *q_d = reinterpret_cast<uint16_t *>(base); base += up(2 * B * eqk);
  uint16_t *k_d = reinterpret_cast<uint16_t *>(base); base += up(2 * B * eqk);
  uint16_t *v_d = reinterpret_cast<uint16_t *>(base); base += up(2 * B * ev);
  uint16_t *b_d = reinterpret_cast<uint16_t *>(base); base += up(2 * B * eb);
  uint16_t *a_d = reinterpret_cast<uint16_t *>(base); base += up(2 * B * ea);
  float *o_d = reinterpret_cast<float *>(base);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint16_t *src_h[5] = {q_h, k_h, v_h, beta_h, alpha_h};
  uint16_t *dst_d[5] = {q_d, k_d, v_d, b_d, a_d};
  const uint64_t per_seq[5] = {eqk, eqk, ev, eb, ea};

  // every sub-batch starts at a multiple of 8 sequences, which keeps all of its pointers 16-byte aligned and
  // all of its arrays whole numbers of 16-byte units
  const uint64_t per = (B / PIPE_CHUNKS + 7) / 8 * 8;
  uint64_t lo[PIPE_CHUNKS + 1];
  for (int c = 0; c < PIPE_CHUNKS; c++) lo[c] = std::min<uint64_t>(B, c * per);
  lo[PIPE_CHUNKS] = B;

  // Inputs: when the host arrays are pinned, mapped into the device and aligned, one gather launch per
  // sub-batch (a few CTAs, which share the device with the kernels of the sub-batch before); otherwise five
  // copies per sub-batch.
  const uint16_t *src_a[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  bool mapped = true;
  for (int i = 0; mapped && i < 5; i++) {
    src_a[i] = aligned16(src_h[i]) ? device_alias(src_h[i]) : nullptr;
    mapped = src_a[i] != nullptr && (2 * B * per_seq[i]) % 16 == 0;
  }

  std::lock_guard<std::mutex> lock(g_pipe_mutex);   // the events below are shared by all callers on a device
  HostPipe *hp = nullptr;
  if ((rc = host_pipe(&hp)) != LQ_OK) return rc;
  // Chained onto the previous call (same staging buffer, stream and layout): the inputs of sub-batch c may be
  // brought in as soon as that call's decode kernel of sub-batch c has read its own - next to that call's
  // window-boundary kernels and copies out - instead of after everything on `stream`.
  const uint64_t layout[5] = {B, Hv, Hqk, (uint64_t)shape->gate, (uint64_t)shape->W};
  const bool chained = hp->chain && hp->stage == stage && hp->stream == st &&
                       std::equal(layout, layout + 5, hp->layout);
  hp->chain = false;                         // set again at the end, if everything was enqueued
  // (the copy-out stream needs no tie at the start: all it does waits for a kernel of this call on `stream`)
  bool ok = chained || (cudaEventRecord(hp->start, st) == cudaSuccess &&    // after everything already on `stream`
                        cudaStreamWaitEvent(hp->s_in, hp->start, 0) == cudaSuccess);
  for (int c = 0; ok && c < PIPE_CHUNKS; c++) {
    const uint64_t b0 = lo[c], nb = lo[c + 1] - lo[c];
    if (nb == 0) continue;
    if (chained) ok = cudaStreamWaitEvent(hp->s_in, hp->done[c], 0) == cudaSuccess;   // (the previous call's record)
    if (!ok) break;
    if (mapped) {
      GatherSegs g;
      for (int i = 0; i < 5; i++) {
        g.src[i] = reinterpret_cast<const uint4 *>(src_a[i] + b0 * per_seq[i]);
        g.dst[i] = reinterpret_cast<uint4 *>(dst_d[i] + b0 * per_seq[i]);
        g.units[i] = static_cast<uint32_t>((2 * nb * per_seq[i] + 15) / 16);
      }
      ok = launch(gather_kernel, sm_count() / 2, 256, 0, hp->s_in, g) == LQ_OK;
    } else {
      for (int i = 0; ok && i < 5; i++)
        ok = cudaMemcpyAsync(dst_d[i] + b0 * per_seq[i], src_h[i] + b0 * per_seq[i], 2 * nb * per_seq[i],
                             cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(hp->in[c], hp->s_in) == cudaSuccess;
  }
  // Kernels on `stream`, sub-batch after sub-batch.  o of a sub-batch is complete after its decode kernel, so
  // its copy to the host starts there, next to the window-boundary kernel, which does not touch o.
  for (int c = 0; ok && c < PIPE_CHUNKS; c++) {
    const uint64_t b0 = lo[c], nb = lo[c + 1] - lo[c];
    if (nb == 0) continue;
    ok = cudaStreamWaitEvent(st, hp->in[c], 0) == cudaSuccess;
    if (!ok) break;
    lq_shape sub = *shape;
    sub.batch = static_cast<int>(nb);
    lq_state ss = *state;
    ss.heads += b0 * Hv * (shape->state_bf16 ? (uint64_t)BF16W_HEAD_BYTES : (uint64_t)head_bytes(shape->r));
    ss.records = static_cast<char *>(ss.records) + b0 * Hv * shape->W * record_floats(diag) * (shape->rec16 ? 2 : 4);
    if (ss.decays) ss.decays += b0 * Hv * shape->W;
    ss.win_pos += b0;
    rc = decode_step_impl(&sub, &ss, q_d + b0 * eqk, k_d + b0 * eqk, v_d + b0 * ev, b_d + b0 * eb, a_d + b0 * ea,
                          o_d + b0 * ev, stream, hp->done[c]);
    if (rc != LQ_OK) break;
    ok = cudaStreamWaitEvent(hp->s_out, hp->done[c], 0) == cudaSuccess &&
         cudaMemcpyAsync(o_h + b0 * ev, o_d + b0 * ev, 4 * nb * ev, cudaMemcpyDeviceToHost, hp->s_out) == cudaSuccess;
  }
  // join: whatever was put on the side streams is waited for by `stream`, also after an error above
  // (`stream` has waited for every copy-in of this call already, sub-batch by sub-batch, unless an error cut the
  // loop above short)
  bool joined = cudaEventRecord(hp->out, hp->s_out) == cudaSuccess && cudaStreamWaitEvent(st, hp->out, 0) == cudaSuccess;
  if (rc != LQ_OK || !ok)
    joined = cudaEventRecord(hp->out, hp->s_in) == cudaSuccess && cudaStreamWaitEvent(st, hp->out, 0) == cudaSuccess &&
             joined;
  if (rc != LQ_OK) return rc;
  if (!ok || !joined) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  hp->chain = true;
  hp->stage = stage;
  hp->stream = st;
  std::copy(layout, layout + 5, hp->layout);
  return LQ_OK;
}

// ---------------------------------------------------------------------------------------------
// Host-buffer decode step without a caller-supplied staging buffer: the staging is this array.
// It is a device object of the library: every GPU that loads the library carries it until exit.  In host
// code the name below is only a handle; the device address comes from cudaGetSymbolAddress, looked up once
// per device and cached.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_stage[LQ_STATIC_STAGE_BYTES];

static lq_status static_stage_address(void **out) {
  constexpr int MAX_DEVICES = 64;
  static std::atomic<void *> cached[MAX_DEVICES];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  void *ptr = cached[dev].load(std::memory_order_acquire);
  if (!ptr) {                                 // first call on this device (it is the current device)
    if (cudaGetSymbolAddress(&ptr, g_static_stage) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return LQ_ERR_CUDA;
    }
    cached[dev].store(ptr, std::memory_order_release);   // two racing first calls store the same address
  }
  *out = ptr;
  return LQ_OK;
}

lq_status lq_decode_step_host_static(const lq_shape *shape, const lq_state *state, const uint16_t *q_h,
                                     const uint16_t *k_h, const uint16_t *v_h, const uint16_t *beta_h,
                                     const uint16_t *alpha_h, float *o_h, lq_stream stream) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  const uint64_t need = lq_decode_stage_bytes(shape);
  if (need > LQ_STATIC_STAGE_BYTES) return LQ_ERR_TOO_LARGE;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;     // before the clearing below is enqueued
  if (!q_h || !k_h || !v_h || !beta_h || !alpha_h || !o_h) return LQ_ERR_NULL;
  void *stage = nullptr;
  if ((rc = static_stage_address(&stage)) != LQ_OK) return rc;
  if (shape->batch == 0) return LQ_OK;
  // The array still holds the previous call's staging.  The inputs are overwritten in full by this call's
  // copies; the output region is cleared, so that rows no kernel writes (sequences with a full window on
  // entry) do not leak an earlier call's results into o_h.  The output region is the last one in the buffer.
  const uint64_t out_bytes = 4ull * shape->batch * shape->heads_v * shape->d_v;
  unsigned char *out_region = static_cast<unsigned char *>(stage) + (need - (out_bytes + 255) / 256 * 256);
  if (cudaMemsetAsync(out_region, 0, out_bytes, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  // always through the staging buffer, so that the cleared output region is what reaches o_h for such rows
  return host_step_impl(shape, state, q_h, k_h, v_h, beta_h, alpha_h, o_h, stage, stream, false);
}

lq_status lq_window_flush(const lq_shape *shape, const lq_state *state, int force, lq_stream stream) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;
  Params p = make_params(shape, state);
  p.force = force ? 1 : 0;
  return launch_boundary<0>(shape, p, reinterpret_cast<cudaStream_t>(stream));
}

lq_status lq_quantize_state(const lq_shape *shape, const float *S, const lq_state *state, lq_stream stream) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if ((rc = check_state(shape, state, false)) != LQ_OK) return rc;
  if ((rc = check_ptrs({S})) != LQ_OK) return rc;
  Params p = make_params(shape, state);
  p.S = const_cast<float *>(S);
  return launch_boundary<1>(shape, p, reinterpret_cast<cudaStream_t>(stream));
}

lq_status lq_dequantize_state(const lq_shape *shape, const lq_state *state, float *S, lq_stream stream) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;
  if ((rc = check_ptrs({S})) != LQ_OK) return rc;
  Params p = make_params(shape, state);
  p.S = S;
  return launch_boundary<2>(shape, p, reinterpret_cast<cudaStream_t>(stream));
}

static lq_status ref_step(const lq_shape *shape, float *S, uint16_t *S16, const uint16_t *q, const uint16_t *k,
                          const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o, lq_stream stream) {
  lq_shape s = *shape;
  s.W = 1; s.r = 0; s.n_iter = 1; s.state_bf16 = 0;      // unused by the baseline
  lq_status rc = check_shape(&s);
  if (rc != LQ_OK) return rc;
  if ((rc = check_ptrs({S ? (const void *)S : (const void *)S16, q, k, v, o})) != LQ_OK) return rc;
  if ((rc = check_scalar_ptrs({beta}, 2)) != LQ_OK) return rc;
  if ((rc = s.gate == LQ_GATE_DIAG ? check_ptrs({alpha}) : check_scalar_ptrs({alpha}, 2)) != LQ_OK) return rc;
  Params p = make_params(&s, nullptr);
  p.S = S; p.S16 = S16; p.q = q; p.k = k; p.v = v; p.beta = beta; p.alpha = alpha; p.o = o;
  const int nh = s.batch * s.heads_v;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const bool diag = s.gate == LQ_GATE_DIAG;
  if (S16) return diag ? launch(ref_kernel<LQ_GATE_DIAG, true>, nh, 256, 0, st, p)
                       : launch(ref_kernel<LQ_GATE_SCALAR, true>, nh, 256, 0, st, p);
  return diag ? launch(ref_kernel<LQ_GATE_DIAG, false>, nh, 256, 0, st, p)
              : launch(ref_kernel<LQ_GATE_SCALAR, false>, nh, 256, 0, st, p);
}

lq_status lq_ref_decode_step_f32(const lq_shape *shape, float *S, const uint16_t *q, const uint16_t *k,
                                 const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                 lq_stream stream) {
  if (!shape) return LQ_ERR_NULL;
  if (!S) return LQ_ERR_NULL;
  return ref_step(shape, S, nullptr, q, k, v, beta, alpha, o, stream);
}

lq_status lq_ref_decode_step_bf16(const lq_shape *shape, uint16_t *S, const uint16_t *q, const uint16_t *k,
                                  const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                  lq_stream stream) {
  if (!shape) return LQ_ERR_NULL;
  if (!S) return LQ_ERR_NULL;
  return ref_step(shape, nullptr, S, q, k, v, beta, alpha, o, stream);
}

static lq_status convert_state(const lq_shape *shape, const lq_state_arrays *arr, const lq_state *state, lq_stream stream,
                               bool import) {
  lq_status rc = check_shape(shape);
  if (rc != LQ_OK) return rc;
  if (shape->state_bf16) return LQ_ERR_UNSUPPORTED;
  if ((rc = check_state(shape, state, true)) != LQ_OK) return rc;
  if (!arr) return LQ_ERR_NULL;
  if ((rc = check_ptrs({arr->codes, arr->col_scale, arr->row_smooth, arr->buf_k, arr->buf_u, arr->buf_a})) != LQ_OK) return rc;
  if (shape->r > 0 && (rc = check_ptrs({arr->comp_k, arr->comp_u})) != LQ_OK) return rc;
  if ((rc = check_scalar_ptrs({arr->win_pos}, 4)) != LQ_OK) return rc;
  Params p = make_params(shape, state);
  const int nh = shape->batch * shape->heads_v;
  const int diag = shape->gate == LQ_GATE_DIAG ? 1 : 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (nh <= 0) return LQ_OK;
  if (import) convert_state_kernel<true><<<nh, 256, 0, st>>>(p, *arr, diag);
  else convert_state_kernel<false><<<nh, 256, 0, st>>>(p, *arr, diag);
  return cudaGetLastError() == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}

lq_status lq_import_state(const lq_shape *shape, const lq_state_arrays *src, const lq_state *dst, lq_stream stream) {
  return convert_state(shape, src, dst, stream, true);
}

lq_status lq_export_state(const lq_shape *shape, const lq_state *src, const lq_state_arrays *dst, lq_stream stream) {
  return convert_state(shape, dst, src, stream, false);
}

lq_status lq_check_device(int *flags) {
  if (!flags) return LQ_ERR_NULL;
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_device_error, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  *flags = v;
  return LQ_OK;
}

lq_status lq_clear_device_flags(void) {
  const int zero = 0;
  if (cudaMemcpyToSymbol(g_device_error, &zero, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return LQ_ERR_CUDA;
  }
  return LQ_OK;
}

uint64_t lq_static_stage_bytes(void) { return LQ_STATIC_STAGE_BYTES; }

}  // extern "C"

// One warp waits, with a limit of a few dozen polls, on a barrier that nothing will ever complete: the wait
// must come back with "gave up", which is reported like in the decode kernel (error flag, bit 3 here).
namespace {
__global__ void bounded_wait_probe_kernel() {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = lq::smem_addr(&bar);
  if (threadIdx.x == 0) lq::mbar_init(b, 1);
  __syncwarp();
  const bool done = lq::mbar_wait<64>(b, 0);
  if (!done && threadIdx.x == 0) atomicOr(&lq::g_device_error, 8);
}
}  // namespace

extern "C" {

lq_status lq_selftest_bounded_wait(lq_stream stream) {
  bounded_wait_probe_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>();
  return cudaGetLastError() == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}

#ifdef LQ_TIMING
// development aid: copies the time stamps of the last four steps to host memory (4 x 2 x 6 x 1024 values)
int lq_debug_timeline(unsigned long long *out) {
  return cudaMemcpyFromSymbol(out, g_timeline, sizeof(unsigned long long) * 4 * 2 * 6 * 1024) != cudaSuccess;
}
// development aid: copies the phase counters to host memory and clears them
int lq_debug_phase_cycles(unsigned long long *out) {
  unsigned long long zero[64] = {0};
  if (cudaMemcpyFromSymbol(out, g_phase_cycles, sizeof(zero)) != cudaSuccess) return 1;
  return cudaMemcpyToSymbol(g_phase_cycles, zero, sizeof(zero)) != cudaSuccess;
}
#endif

int lq_decode_launches(const lq_shape *shape) { return check_shape(shape) == LQ_OK && shape->batch > 0 ? 2 : 0; }

const char *lq_status_string(lq_status status) {
  switch (status) {
    case LQ_OK: return "ok";
    case LQ_ERR_NULL: return "null pointer";
    case LQ_ERR_SHAPE: return "invalid shape";
    case LQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case LQ_ERR_UNSUPPORTED: return "shape not supported";
    case LQ_ERR_CUDA: return "CUDA runtime error";
    case LQ_ERR_TOO_LARGE: return "request exceeds the built-in scratch buffer";
  }
  return "unknown status";
}

int lq_version(void) { return 7; }

}  // extern "C"
