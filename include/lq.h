/*
 * lq.h - C boundary of the B200 (sm_100a) per-window 8-bit decode step for
 * Gated DeltaNet (scalar gate) and Kimi Delta Attention (per-channel gate)
 * recurrent states.
 *
 * One value head owns a state S in R^{d_k x d_v} (Sec. 3.1, Eq. 1; row index =
 * key channel, column index = value channel, readout o = S^T q).  Between
 * window boundaries the state is held as
 *     S_l = Gamma_{1:l} [ C (Z/127) B + Kc Uc^T ] + sum_j Gamma_{j+1:l} kt_j u_j^T      (Eq. 7)
 * with Z the 8-bit codes, B the per-value-channel scale, C = Diag(c) the
 * per-key-row smoothing scale (Sec. 3.4), (Kc, Uc) the r fp16 Compensator
 * Tokens (Sec. 3.3) and (alpha_j, kt_j, u_j) the buffered records of the
 * tokens decoded since the boundary (Sec. 3.2, Eq. 3).
 *
 * Conventions for every entry point
 *  - All pointers are DEVICE pointers owned by the caller unless a parameter
 *    is documented as a host pointer.  Arrays are dense, row-major, in the
 *    layouts given below, and must be 16-byte aligned.
 *  - The library allocates no device memory and never synchronises: work is
 *    enqueued on `stream` and the call returns.  The lq_shape and lq_state
 *    structs themselves are read on the host during the call only.
 *  - bf16 and fp16 values travel as their 16-bit patterns (uint16_t).
 *  - Errors are reported through the return value; nothing aborts or throws.
 *    Argument errors are detected before anything is enqueued (the host-buffer
 *    entry points included).
 *  - Arithmetic is IEEE binary32.  Sums over a channel index are taken in a
 *    fixed order (blocks of eight consecutive terms; inside a block the
 *    even-numbered and the odd-numbered terms are two chains of fused
 *    multiply-adds that are added at the end; block results combined as a
 *    balanced binary tree over the block index, neighbours first), and the
 *    code-matrix term of the readout is an exact integer sum, so results do
 *    not depend on the launch configuration and are reproducible bit for bit.
 *  - Supported shapes: d_k = d_v = 128, 1 <= W <= 64, 0 <= r <= 16,
 *    n_iter >= 1, heads_v a multiple of heads_qk.  Anything else returns
 *    LQ_ERR_UNSUPPORTED.
 */
#ifndef LQ_H_
#define LQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LQ_OK = 0,
  LQ_ERR_NULL = 1,        /* a required pointer is null                         */
  LQ_ERR_SHAPE = 2,       /* a dimension is non-positive or inconsistent        */
  LQ_ERR_ALIGN = 3,       /* a pointer is not 16-byte aligned                   */
  LQ_ERR_UNSUPPORTED = 4, /* valid request outside the supported shapes         */
  LQ_ERR_CUDA = 5,        /* the CUDA runtime reported an error on launch/copy  */
  LQ_ERR_TOO_LARGE = 6    /* the request does not fit the library's built-in scratch buffer */
} lq_status;

typedef enum {
  LQ_GATE_SCALAR = 0, /* GDN: D_t = alpha_t I;       alpha is [B,Hv]       */
  LQ_GATE_DIAG = 1    /* KDA: D_t = Diag(alpha_t);   alpha is [B,Hv,d_k]   */
} lq_gate;

/* CUDA stream handle (a cudaStream_t); null is the default stream. */
typedef struct CUstream_st *lq_stream;

typedef struct {
  int batch;    /* B: sequences                                                   */
  int heads_v;  /* Hv: value heads per sequence, one state each                   */
  int heads_qk; /* Hqk: query/key heads; value head h reads q/k head h/(Hv/Hqk)   */
  int d_k, d_v; /* state is d_k x d_v                                             */
  int W;        /* window length (the paper's p)                                  */
  int r;        /* Compensator Tokens per state                                   */
  int n_iter;   /* rounds of the power iteration at a boundary (1 is the default of */
                /* the binding).  All r vectors are iterated together: T = S W,     */
                /* orthonormalise, W = S^T T, orthonormalise, ...; column h of W    */
                /* starts from the u of the (h+1)-th newest buffered record, or     */
                /* from Walsh function h where there is no such record              */
  int gate;     /* lq_gate                                                        */
  int smooth;   /* 1: residual smoothing (Sec. 3.4); 0: c = 1 (ablation)          */
  int delta;    /* 1: delta rule, the correction reads the state back with          */
                /* b = alpha (.) k (DeltaNet, Gated DeltaNet, KDA);                 */
                /* 0: b = 0, u = v (the other instances of the paper's Table 4:     */
                /* linear attention, RetNet, Mamba2 with the scalar gate; GLA,      */
                /* RWKV6, HGRN2 with the diagonal gate; pass beta = 1 for k~ = k)   */
  int rec16;    /* 1: the record buffer holds fp16 values, as in the paper's storage      */
                /* accounting (kt, u and the diagonal gate's alpha are rounded, with       */
                /* saturation, when a record is appended; the scalar gate's decays stay    */
                /* fp32; `o` of the appending token uses the unrounded u); 0: fp32 records */
  int state_bf16; /* 1: "per-window BF16", the -w baseline of the paper's Fig. 3 and Table 2: the    */
                /* boundary state is the dense state rounded to bfloat16 (nearest even) once per  */
                /* window, with no scale, smoothing or compensator; needs r = 0 and smooth = 0;   */
                /* the readout is S0^T x in binary32 in the fixed summation order.  0: the 8-bit  */
                /* representation of Eq. 7                                                        */
} lq_shape;

/*
 * Window representation of B x Hv states, laid out for bulk transfers: everything that is read once per
 * token and head is contiguous.
 *
 * heads: one block of lq_head_bytes(shape) bytes per (sequence, value head), [B,Hv] blocks back to back:
 *     offset 0                        codes      int8 [d_v][d_k]  Z^T: the code of S[i][j] sits at [j][i]
 *                                                (value-channel major, so that the key index is contiguous);
 *                                                symmetric, in [-127,127]
 *     + d_k*d_v                       col_scale  fp32 [d_v]       step of the code per value channel, B_j/127:
 *                                                dequant(Z)_ij = Z_ij * col_scale_j  (Appendix B.3)
 *     + 4*d_v                         row_smooth fp32 [d_k]       c > 0 (Sec. 3.4)
 *     + 4*d_k                         comp_k     fp16 [r][d_k]    unit-length key side of the compensators
 *     + 2*r*d_k                       comp_u     fp16 [r][d_v]    value side (carries the magnitude)
 *   (17408 + 512 r bytes at d_k = d_v = 128: 19456 for r = 4, i.e. 1.19 bytes per state element.)
 *   With shape.state_bf16 the block is instead   state  bf16 [d_v][d_k]   S0^T: S0[i][j] sits at [j][i]
 *   (32768 bytes).
 *
 * records: one row of lq_record_floats(shape) values (fp32, or fp16 with shape.rec16) per buffered record, [B,Hv,W] rows:
 *     kt[d_k] | u[d_v]                write key kt = beta*k and correction u = v - S^T(alpha.k)  (Eq. 3)
 *     | alpha[d_k]                    diagonal gate only: the record's decay
 * decays: scalar gate only, fp32 [B,Hv,W]: the decay of each buffered record (ignored for the diagonal gate).
 * win_pos: int32 [B], records buffered per sequence, 0..W-1 between calls.  Bits 16 and up are used as a
 *     scratch counter while a call runs and are zero again when it has finished.
 * work: optional (may be null): int32 [LQ_WORK_WORDS], all zero when the state is created and zero again after
 *     every call.  With it, the decode kernel of lq_decode_step hands out the heads of its last, partial round
 *     (B*Hv heads over the CTAs that are resident at once) to the CTAs that get there first, instead of giving
 *     every CTA the same number of heads: on a GPU whose memory system does not serve all SMs alike, equal shares
 *     do not take equal time.  Results are the same bit for bit either way.  Sub-batches of one state that are
 *     addressed by pointer offset may share one `work` as long as their calls do not run at the same time (calls
 *     in one stream never do).  After a call that returned LQ_ERR_CUDA the words are to be zeroed again (and the
 *     state restored from a checkpoint: a step that was enqueued in part leaves neither valid).
 */
#define LQ_WORK_WORDS 8
typedef struct {
  uint8_t *heads;
  void *records;   /* float rows, or (shape.rec16) fp16 rows of the same element counts */
  float *decays;
  int32_t *win_pos;
  int32_t *work;
} lq_state;

/* Size in bytes of one head block, and the number of fp32 values in one record row (0 for an invalid shape). */
uint64_t lq_head_bytes(const lq_shape *shape);
uint64_t lq_record_floats(const lq_shape *shape);

/*
 * One decode token for every (sequence, value head): Eq. 10 (the readout of the smoothed, compensated
 * window representation) applied to alpha.k gives the correction u of Eq. 3, applied to alpha.q gives
 * the output through S_l^T q = S_{l-1}^T (alpha.q) + u (kt^T q); the record (alpha, kt, u) is appended
 * to the buffer and win_pos advances.  A sequence whose window becomes full (win_pos reaches W) is
 * taken through the boundary in the same call, as Eq. 4 prescribes: see lq_window_flush.
 *   q, k  : bf16 [B,Hqk,d_k]     v : bf16 [B,Hv,d_v]     beta : bf16 [B,Hv]
 *   alpha : bf16 [B,Hv] or [B,Hv,d_k], the decay multiplier itself (not its logarithm)
 *   o     : fp32 [B,Hv,d_v], written
 * A sequence that enters with win_pos >= W (possible only if the caller set it) gets no token: its `o`
 * rows are not written and nothing is appended; with win_pos == W it is taken through the boundary by
 * this call like by lq_window_flush.
 * Calls on the same state must be ordered by the stream.
 */
lq_status lq_decode_step(const lq_shape *shape, const lq_state *state, const uint16_t *q, const uint16_t *k,
                         const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o, lq_stream stream);

/*
 * lq_decode_step for a measuring harness: identical work, and in addition the CUDA event `event_between`
 * (a cudaEvent_t created by the caller; may be null) is recorded on `stream` between the decode kernel and
 * the window-boundary kernel, so that the two can be timed separately.
 */
lq_status lq_decode_step_profiled(const lq_shape *shape, const lq_state *state, const uint16_t *q, const uint16_t *k,
                                  const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                  lq_stream stream, void *event_between);

/*
 * Same as lq_decode_step, but the token's inputs and the output live in HOST memory (pinned memory makes
 * the copies asynchronous): q_h, k_h, v_h, beta_h, alpha_h are copied into the device staging buffer
 * `stage` on `stream`, the step runs, and `o` is copied to o_h.  `stage` is a device buffer of at least
 * lq_decode_stage_bytes(shape) bytes, 16-byte aligned, owned by the caller.  The host arrays must stay
 * valid until the stream has passed the call.
 */
lq_status lq_decode_step_host(const lq_shape *shape, const lq_state *state, const uint16_t *q_h,
                              const uint16_t *k_h, const uint16_t *v_h, const uint16_t *beta_h,
                              const uint16_t *alpha_h, float *o_h, void *stage, lq_stream stream);
/*
 * lq_decode_step_host with the host<->device transfers overlapped with the kernels.  (The paper's path
 * starts and ends in device memory; this is a convenience of the library for callers whose tokens arrive in
 * host memory.)  The batch is cut into two sub-batches of whole sequences.  The inputs of both are brought in
 * on a copy-in stream, so the second sub-batch arrives while the first is computed; o of a sub-batch is
 * complete after its decode kernel and is copied out on a copy-out stream while the window-boundary kernel of
 * that sub-batch and the next sub-batch run.  The two side streams are created per device at the first call
 * (make that call outside any stream capture) and are tied to `stream` by events on both sides: the call
 * starts after everything already enqueued on `stream`, and anything enqueued on `stream` afterwards starts
 * after the last copy.  Same arguments, staging size, results and error codes as lq_decode_step_host; use
 * pinned host memory, otherwise nothing overlaps.  Batches below sixteen sequences take the unpipelined path.
 * Calls from several host threads are serialised inside the library while they enqueue.
 *
 * Consecutive calls with the same `stage`, `stream` and shape chain onto each other: the inputs of sub-batch c of
 * the later call are brought in as soon as the earlier call's decode kernel of sub-batch c has consumed its own,
 * i.e. next to the earlier call's window-boundary kernels and copies out, and possibly before other work that
 * was enqueued on `stream` in between.  So the host input arrays must hold their final values when the call is
 * made (not merely when `stream` reaches it), and between such calls `stage` belongs to the library.  A call of
 * lq_decode_step_host or lq_decode_step_host_static, another `stage` or another stream ends the chain; the next
 * pipelined call is then ordered after everything on `stream` again.  Outputs are always stream-ordered: what is
 * enqueued on `stream` after a call finds o_h complete.
 *
 * Both host-buffer entry points read the inputs with ONE gather launch (per sub-batch) instead of five copies
 * when all input arrays are pinned, mapped into the device (cudaHostAlloc / cudaHostRegister memory under
 * unified addressing) and 16-byte aligned with sizes that are multiples of 16 bytes; lq_decode_step_host
 * then also lets the decode kernel write o straight into the host array.  Otherwise they fall back to
 * cudaMemcpyAsync.  The results are the same either way.
 */
lq_status lq_decode_step_host_pipelined(const lq_shape *shape, const lq_state *state, const uint16_t *q_h,
                                        const uint16_t *k_h, const uint16_t *v_h, const uint16_t *beta_h,
                                        const uint16_t *alpha_h, float *o_h, void *stage, lq_stream stream);
/* Bytes of device staging lq_decode_step_host needs for `shape` (0 if the shape is invalid). */
uint64_t lq_decode_stage_bytes(const lq_shape *shape);

/*
 * lq_decode_step_host for callers that cannot hand over a staging buffer because they cannot allocate one.
 * (The paper has no counterpart: this is a convenience of the library.)
 *
 * Who this is for: a serving process that gave all of the device's memory to its own pools when it started
 * has nothing left for cudaMalloc to return, and a decode loop that must never stall cannot afford
 * cudaMalloc/cudaFree either, since both may synchronise the whole device.  Such a caller still owns the
 * host arrays and the lq_state, but has nowhere to put the few megabytes of staging that the host-buffer
 * path needs.  Here the staging lives inside the library, in a fixed device array of
 * LQ_STATIC_STAGE_BYTES bytes that every GPU that loads the library keeps reserved until the process
 * exits.  The call itself allocates and frees nothing, on the device or through any library.
 *
 * Same arguments and behaviour as lq_decode_step_host without `stage`, with these differences:
 *  - lq_decode_stage_bytes(shape) must not exceed LQ_STATIC_STAGE_BYTES, otherwise LQ_ERR_TOO_LARGE is
 *    returned and nothing is enqueued (16 MiB covers 256 sequences x 32 heads, the benchmark batch).
 *  - The first call on each device looks up the device address of the built-in array (with that device
 *    current).  Make that first call outside any stream capture.
 *  - The array is shared by all calls and keeps what the previous call left in it.  The output staging is
 *    therefore cleared at the start of every call: rows of o_h that belong to sequences which get no token
 *    (win_pos >= W on entry) come back as zeros.
 *  - Because the array is shared, two calls whose work overlaps on the GPU (different streams, or different
 *    host threads) race on it.  Order them on one stream, or use lq_decode_step_host with separate buffers.
 */
#define LQ_STATIC_STAGE_BYTES (16u << 20)
lq_status lq_decode_step_host_static(const lq_shape *shape, const lq_state *state, const uint16_t *q_h,
                                     const uint16_t *k_h, const uint16_t *v_h, const uint16_t *beta_h,
                                     const uint16_t *alpha_h, float *o_h, lq_stream stream);

/*
 * Window boundary (Secs. 3.2-3.4): for every sequence with win_pos == W, or, when force != 0, with
 * win_pos > 0, rebuild the dense state from the window representation (Eq. 7), refit the r Compensator
 * Tokens by power iteration and remove them (Eqs. 5-6), recompute the smoothing scales from the
 * residual, requantize it to 8 bits, and set win_pos = 0.  Other sequences are not touched.
 */
lq_status lq_window_flush(const lq_shape *shape, const lq_state *state, int force, lq_stream stream);

/*
 * Start a window from dense states: S fp32 [B,Hv,d_k,d_v] (read only) is split into compensators,
 * smoothing scales and 8-bit codes exactly as at a window boundary; win_pos is set to 0 for all B
 * sequences.  The record buffers are not read or written.
 */
lq_status lq_quantize_state(const lq_shape *shape, const float *S, const lq_state *state, lq_stream stream);

/*
 * The dense state the window representation currently stands for, all buffered records applied (Eq. 7
 * with l = win_pos): written to S fp32 [B,Hv,d_k,d_v].  The state is not modified.
 */
lq_status lq_dequantize_state(const lq_shape *shape, const lq_state *state, float *S, lq_stream stream);

/*
 * The window representation as separate arrays in the paper's notation and orientation (Sec. 3.1: S is d_k x d_v;
 * Appendix B.3 for Z and B; Sec. 3.4 for c; Sec. 3.3 for the compensators; Eq. 3 for the records), for callers
 * that hold or want the state that way instead of in the packed head blocks above.  All arrays dense, row-major,
 * device memory, 16-byte aligned:
 *   codes      int8 [B,Hv,d_k,d_v]   Z (NOT transposed)
 *   col_scale  fp32 [B,Hv,d_v]       step of the code per value channel, B_j / 127
 *   row_smooth fp32 [B,Hv,d_k]       c
 *   comp_k     fp16 [B,Hv,r,d_k]     comp_u  fp16 [B,Hv,r,d_v]      (null when r = 0)
 *   buf_k      fp32 [B,Hv,W,d_k]     write keys beta*k of the buffered records
 *   buf_u      fp32 [B,Hv,W,d_v]     corrections u
 *   buf_a      fp32 [B,Hv,W] (scalar gate) or [B,Hv,W,d_k] (diagonal gate): the records' decays
 *   win_pos    int32 [B]
 * lq_import_state fills `dst` from the arrays, lq_export_state the arrays from `src`; both copy all W record
 * slots whatever win_pos says.  With shape.rec16 the records are narrowed to fp16 on import (nearest even,
 * saturating) and widened on export.  Not available with shape.state_bf16 (LQ_ERR_UNSUPPORTED).
 */
typedef struct {
  int8_t *codes;
  float *col_scale;
  float *row_smooth;
  uint16_t *comp_k;
  uint16_t *comp_u;
  float *buf_k;
  float *buf_u;
  float *buf_a;
  int32_t *win_pos;
} lq_state_arrays;
lq_status lq_import_state(const lq_shape *shape, const lq_state_arrays *src, const lq_state *dst, lq_stream stream);
lq_status lq_export_state(const lq_shape *shape, const lq_state *src, const lq_state_arrays *dst, lq_stream stream);

/*
 * Speed and accuracy baselines: the same token on an unquantized dense state (Eq. 1 with the GDN / KDA
 * coefficients of Table 4), read and written in full every token.  S is [B,Hv,d_k,d_v], fp32 or bf16
 * (rounded to nearest even after every token, the "BF16 per-step" setting); o is computed from the
 * updated state before it is rounded.  Only batch, heads_v, heads_qk, d_k, d_v and gate of `shape` are used.
 */
lq_status lq_ref_decode_step_f32(const lq_shape *shape, float *S, const uint16_t *q, const uint16_t *k,
                                 const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                 lq_stream stream);
lq_status lq_ref_decode_step_bf16(const lq_shape *shape, uint16_t *S, const uint16_t *q, const uint16_t *k,
                                  const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, float *o,
                                  lq_stream stream);

/*
 * Device-side error flags of the current device (0 = none), written to *flags (a host pointer).  Waits inside
 * the kernels are bounded; bit 0 is set when a decode warp gave up waiting for its asynchronous copies.  After
 * that, neither the outputs of that launch NOR THE STATE it worked on are valid (records may be missing or
 * half written): restore the state from a checkpoint.  Bits 1 and 2 belong to the optional fused step kernel
 * (gave up waiting for decode work / more heads than it can track), bit 3 to lq_selftest_bounded_wait.
 * The flags stay set until lq_clear_device_flags is called.  Both calls synchronise the device.
 */
lq_status lq_check_device(int *flags);
lq_status lq_clear_device_flags(void);

/*
 * Self test of the give-up path of the bounded waits (no passage of the paper): launches one warp that
 * waits, with a limit of 64 polls, on a barrier nothing completes.  The wait returns "gave up", the warp sets
 * bit 3 of the error flags and exits; the context stays usable.  Read the flag with lq_check_device and clear
 * it with lq_clear_device_flags.
 */
lq_status lq_selftest_bounded_wait(lq_stream stream);

/* LQ_STATIC_STAGE_BYTES as the loaded library was built with (for bindings that cannot read the macro). */
uint64_t lq_static_stage_bytes(void);

/* Kernels one lq_decode_step call launches for `shape` (used to report launch counts). */
int lq_decode_launches(const lq_shape *shape);

const char *lq_status_string(lq_status status);
int lq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LQ_H_ */
