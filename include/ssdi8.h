/* ssdi8.h -- C ABI of the B200 (sm_100a) INT8 State Space Duality layer.
 *
 * The library computes the forward pass of one quantised Mamba-2 SSD layer
 * (SSDi8, Algorithm 2 with the INT8 path of Section 4.2) and its single-token
 * recurrent step.  Symbols follow the paper: batch B (here `batch`), length L,
 * heads H, head dimension P, state dimension N, groups G, chunk length l
 * (here Q = `chunk`), c = L / Q chunks, D = H * P channels, g(h) = h / (H / G).
 *
 * Conventions for every entry point
 *  - All pointers are DEVICE pointers unless the comment says "host".  The
 *    caller owns every buffer and the library allocates no device memory.  It keeps
 *    no mutable state between calls, with three exceptions, each stated again at its
 *    entry point: per device, the result of the architecture check (every call);
 *    the address of the built-in scratch (ssdi8_chunk_scan_fwd_static); two copy
 *    streams and their events (ssdi8_layer_fwd_host, created at the first call on
 *    a device and kept for the life of the process).  All three are
 *    filled under a lock, so first calls may come from several threads at once.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls are asynchronous on that stream.
 *  - The return value reports everything that can be checked on the host
 *    before launch (null pointers, unsupported shapes, alignment, short
 *    workspace, wrong device architecture, launch failure).  Nothing throws
 *    and nothing aborts.  A condition detected on the device (a bounded wait
 *    that ran out) is written to the caller's `status` word, to be read after
 *    synchronising the stream.
 *  - Tensors are dense, row-major, last axis contiguous.
 *  - Supported shapes: P = 64, N in {64, 128}, Q in {64, 128, 256}, L % Q = 0,
 *    H % G = 0; otherwise SSDI8_ERR_SHAPE.
 *  - Every int8 code the library produces lies in [-127, 127].
 *  - Results are deterministic: no floating-point atomics in any result.
 *
 * Arithmetic that decides an integer code is carried out in IEEE binary32 with
 * round-to-nearest-even, in the operation order written in each comment below
 * (fmul, fsub, fdiv, fmaf are single correctly rounded operations; rne rounds
 * half to even and the result is then saturated to [-127, 127]).  exp32 is the
 * library's binary32 exponential: n = rint(x * 0x3FB8AA3B), r = fmaf(n,
 * -0x3F317200, x), r = fmaf(n, -0x35BFBE8E, r), degree-7 Taylor polynomial in r
 * by Horner with fmaf, result scaled by 2^n; 0 for x < -80.
 */
#ifndef SSDI8_H_
#define SSDI8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t ssdi8_status_t;
enum {
  SSDI8_OK = 0,
  SSDI8_ERR_NULL = -1,           /* a required pointer is NULL                        */
  SSDI8_ERR_SHAPE = -2,          /* unsupported or inconsistent dimensions            */
  SSDI8_ERR_ALIGN = -3,          /* a pointer is not 16-byte aligned                  */
  SSDI8_ERR_WORKSPACE = -4,      /* workspace shorter than ssdi8_workspace_bytes()    */
  SSDI8_ERR_ARCH = -5,           /* current device is not compute capability 10.0     */
  SSDI8_ERR_CUDA = -6,           /* a CUDA runtime call or a launch failed            */
  SSDI8_ERR_DEVICE_TIMEOUT = -7, /* written to *status by a kernel whose wait ran out */
  SSDI8_ERR_UNSUPPORTED = -8     /* a flag or mode that is not implemented            */
};

typedef struct {
  int32_t batch, seqlen, nheads, headdim, dstate, ngroups, chunk;
} ssdi8_dims_t;

/* module selection bits of ssdi8_chunk_scan_fwd's flags (Algorithm 2's modules) */
enum {
  SSDI8_PHASE_CUMSUM = 1u << 8,
  SSDI8_PHASE_BMM = 1u << 9,
  SSDI8_PHASE_CHUNK_STATE = 1u << 10,
  SSDI8_PHASE_STATE_PASSING = 1u << 11,
  SSDI8_PHASE_SCAN = 1u << 12,
  SSDI8_PHASE_ALL = 0x1f00u
};

/* operand format bit of ssdi8_chunk_scan_fwd's flags: the paper's own ChunkScan2 (Section 4.2;
 * Algorithm 2, module 6) instead of the per-row int8 re-quantisation of the masked operand:
 *   M16[i,j] = half(s_cb CBq[i,j] dt_j exp(cs_i - cs_j)), j <= i   (FP16, CB's scale fused into the LUT)
 *   y_diag   = s_x sum_j M16[i,j] xq[j,p]      (FP16 tensor-core MMA, FP32 accumulation; X enters as
 *                                               the exact FP16 image of its int8 codes)
 * computed with one factor per 16-token sub-block as below (own sub-block: running product of the
 * per-token decays; earlier: woff_j f), in binary32 before the rounding to FP16, so a value may
 * differ from the definition by one FP16 unit in the last place.  The codes of x are expanded to FP16
 * on the chip; the mode needs no workspace of its own.  Not combinable with the scan taps. */
enum { SSDI8_FLAG_FP16_OPERAND = 1u << 0 };

/* state format bit of ssdi8_chunk_scan_fwd's flags */
enum { SSDI8_FLAG_INT8_STATE = 1u << 1 };

/* time-step bit of ssdi8_chunk_scan_fwd's flags: `dt` holds the raw time step and ChunkCumsum starts, as
 * Algorithm 2 module 1 does, from dt = softplus(dt_raw + dt_bias[h]) (dt_bias = NULL: no bias).  The
 * value is formed in binary64, each step one correctly rounded operation, and rounded to binary32 once:
 *   v = (double) fadd(dt_raw, dt_bias);  a = |v|
 *   u = exp(-a): n = rint(-a LOG2E), r = fma(n, -LN2_HI, -a), r = fma(n, -LN2_LO, r) with
 *       LOG2E = 0x1.71547652b82fep+0, LN2_HI = 0x1.62e42fee00000p-1, LN2_LO = 0x1.a39ef35793c76p-33,
 *       degree-13 Taylor polynomial in r by Horner with fma, times 2^n through the exponent field; 0 if a > 700
 *   s = u / (2 + u), z = s s, q = 1 + z/3 + ... + z^13/27 by Horner with fma, lp = (2 s) q   (= log(1 + u))
 *   dt = (float)(max(v, 0) + lp)
 * which equals the correctly rounded softplus in all but about one value in ten million. */
enum { SSDI8_FLAG_DT_SOFTPLUS = 1u << 4 };

/* output format bits (at most one): y is written as 16-bit elements, the paper's own output
 * format being FP16 (Algorithm 2 keeps Y in half precision); default is binary32 */
enum { SSDI8_FLAG_Y_FP16 = 1u << 2, SSDI8_FLAG_Y_BF16 = 1u << 3 };

/* host, pure: static string for a status code */
const char* ssdi8_status_string(ssdi8_status_t s);

/* host, pure: bytes of scratch ssdi8_chunk_scan_fwd / ssdi8_calibrate need for
 * these dimensions (0 if the dimensions are unsupported). */
size_t ssdi8_workspace_bytes(const ssdi8_dims_t* dims, uint32_t flags);

/* Activation quantiser (Eq. 1): uniform symmetric 8-bit, one step size per
 * channel of the view in[R][Ch][I]  (x: R = B*L, Ch = D, I = 1;  B and C,
 * quantised once on the group axis before any broadcast to heads, Section 4.2
 * "Quantization of B,C": R = B*L, Ch = G, I = N).
 *   alpha = fdiv(absmax, 127)  (1 if the channel is all zero)
 *   q     = rne(fdiv(v, alpha)) saturated
 * mode 0 static:    read scale[Ch], write out.
 * mode 1 calibrate: write scale[Ch] from this tensor, then write out.
 * mode 2 observe:   scale[Ch] = max(scale[Ch], alpha of this tensor); `out`
 *                   may be NULL (nothing is quantised then).
 * in, out: 16-byte aligned; I == 1 or I % 4 == 0; (Ch * I) % 4 == 0. */
ssdi8_status_t ssdi8_quantize_act(const float* in, int64_t R, int64_t Ch, int64_t I,
                                  float* scale, int32_t mode, int8_t* out, void* stream);

/* Entry quantiser: the convolution output of a Mamba-2 block is one tensor xBC [T][D + 2 G N]
 * (x, B, C along the last axis; T = B*L, D = H*P).  One pass writes xq [T][D], Bq [T][G*N] and
 * Cq [T][G*N] with static step sizes (Eq. 1, q = rne(fdiv(float(v), alpha)) saturated): x per
 * channel (s_x[D]), B and C per group (s_B[G], s_C[G]), i.e. B and C are quantised once on the
 * group axis at layer entry and the int8 tensors are reused by every module (Section 4.2,
 * "Quantization of B,C").  dtype of xBC: 0 = fp32, 1 = fp16, 2 = bf16 (the conversion to binary32
 * is exact).  D % 4 == 0, N % 4 == 0; xBC, s_x and the outputs 16-byte aligned. */
ssdi8_status_t ssdi8_quantize_entry(const void* xBC, int32_t dtype, int64_t T, int32_t D, int32_t G,
                                    int32_t N, const float* s_x, const float* s_B, const float* s_C,
                                    int8_t* xq, int8_t* Bq, int8_t* Cq, void* stream);

typedef struct {
  /* layer inputs */
  const int8_t* xq;        /* [B,L,H,P]  per-channel codes of X                         */
  const int8_t* Bq;        /* [B,L,G,N]  per-group codes of B                           */
  const int8_t* Cq;        /* [B,L,G,N]  per-group codes of C                           */
  const float* s_x;        /* [H*P] step sizes of xq                                    */
  const float* s_B;        /* [G]                                                       */
  const float* s_C;        /* [G]                                                       */
  const float* dt;         /* [B,L,H] time step, already positive (after softplus), or raw with SSDI8_FLAG_DT_SOFTPLUS */
  const float* A;          /* [H] decay rate, negative                                  */
  const float* D;          /* [H] skip weight, or NULL                                  */
  const float* corr;       /* [H*P] per-channel mean correction (Eq. 8), or NULL        */
  /* static step sizes of the internal int8 tensors (from ssdi8_calibrate) */
  const float* s_xs;       /* [H*P] Q(X_scaled), Eq. 3                                  */
  const float* s_cb;       /* [G]   Q(CB)                                               */
  const float* s_h;        /* [H*P] Q(State), Eq. 4; one scale for all chunks           */
  const float* init_state; /* [B,H,P,N] state before the first token, or NULL (zeros)   */
  /* outputs */
  float* y;                /* [B,L,H,P]                                                  */
  float* final_state;      /* [B,H,P,N] state after the last token, or NULL             */
  int32_t* status;         /* 1 word, or NULL: 0 or an SSDI8_ERR_* written by a kernel   */
  /* optional taps of the intermediate tensors (tests); each may be NULL */
  float* tap_cs;           /* [B,H,c,Q]   chunk-local cumulative sum of dt*A            */
  int32_t* tap_acc_cb;     /* [B,c,G,Q,Q] INT32 C B^T, entries with j <= i              */
  int8_t* tap_CBq;         /* [B,c,G,Q,Q] its int8 codes, entries with j <= i           */
  int8_t* tap_Xsq;         /* [B,L,H,P]   Q(X_scaled)                                   */
  int32_t* tap_acc_st;     /* [B,c,H,P,N] INT32 chunk state                             */
  float* tap_loc;          /* [B,c,H,P,N] chunk-local state, fp32                       */
  float* tap_prev;         /* [B,c,H,P,N] state entering chunk k                        */
  int8_t* tap_hq;          /* [B,c,H,P,N] its int8 codes                                */
  int32_t* tap_acc_off;    /* [B,L,H,P]   INT32 C h                                     */
  float* tap_rowmax;       /* [B,L,H]     absmax of each row of the masked operand      */
  int8_t* tap_Mq;          /* [B,c,H,Q,Q] int8 masked operand, zero above the diagonal  */
  int32_t* tap_acc_diag;   /* [B,L,H,P]   INT32 Mq x                                    */
  /* with SSDI8_FLAG_DT_SOFTPLUS: bias added to the raw time step before the softplus, or NULL */
  const float* dt_bias;    /* [H]                                                        */
} ssdi8_fwd_args_t;

/* SSD layer forward (Algorithm 2) from int8 x, B, C to fp32 y and final state.
 *  ChunkCumsum   (with SSDI8_FLAG_DT_SOFTPLUS first dt = softplus(dt + dt_bias), see the flag)
 *                cs[k,i] = (float) sum_{i'<=i} (double)dt * (double)A, in token order;
 *                Gamma_k = exp32(cs[k,Q-1])                         (Decay_pass, Eq. 5)
 *  ChunkBMM      acc_cb[i,j] = sum_n Cq[i,n] Bq[j,n]  per (b, chunk, group), INT32;
 *                CBq = rne(fmul(float(acc_cb), fdiv(fmul(s_C, s_B), s_cb)))
 *  ChunkState    sparse-aware reformulation, Eq. 3:
 *                LUT_state[i] = fmul(dt_i, exp32(fsub(cs_last, cs_i)))
 *                Xs_q[i,p] = rne(fmul(fmul(float(xq[i,p]), fdiv(s_x, s_xs)), LUT_state[i]))
 *                acc_st[p,n] = sum_i Xs_q[i,p] Bq[i,n], INT32;
 *                loc = fmul(float(acc_st), fmul(s_xs, s_B))          (Eq. 4 rescale)
 *  StatePassing  S_k = fmaf(Gamma_k, S_{k-1}, loc_k), S_{-1} = init_state (Eq. 6), fp32;
 *                hq[k] = rne(fmul(S_{k-1}, fdiv(1, s_h)))
 *  ChunkScan1    acc_off[i,p] = sum_n Cq[i,n] hq[k][p,n], INT32;
 *                y_off = exp(cs_i) s_C s_h acc_off   (decay only; no dt factor)
 *  ChunkScan2    the masked operand CB o LUT_scan2 (LUT_scan2[i,j] = dt_j exp(cs_i - cs_j),
 *                j <= i) is re-quantised per output row so that its product with int8 X is
 *                an integer GEMM.  With sub-blocks of SB = 16 tokens and je the last
 *                column of the sub-block of j:
 *                  same sub-block : running product of the per-token decays
 *                                   a_m = exp32(fsub(cs_m, cs_{m-1})): E[i,i] = 1,
 *                                   E[i,j] = fmul(E[i,j+1], a_{j+1}); w = fmul(dt_j, E[i,j]), f = 1
 *                  earlier block  : w = fmul(dt_j, exp32(fsub(cs_je, cs_j))),
 *                                   f = fmul(exp32(fsub(cs_i, cs_pe)), exp32(fsub(cs_pe, cs_je))), pe the last
 *                                   token of the sub-block before the row's own (the second factor
 *                                   depends on the two sub-blocks only: ChunkCumsum tabulates it)
 *                  t = fmul(float(CBq[i,j]), w)
 *                  rowmax_i = max over sub-blocks of fmul(max_j |t|, f)
 *                  inv_i = rowmax_i >= 1e-30 ? fdiv(127, rowmax_i) : 0
 *                  Mq[i,j] = rn(t * fmul(f, inv_i)): the exact product rounded once to the nearest
 *                            integer, ties to even (the low bits of fmaf(t, fmul(f, inv_i), 1.5 * 2^23))
 *                acc_diag[i,p] = sum_{j<=i} Mq[i,j] xq[j,p], INT32;
 *                y_diag = (s_cb rowmax_i / 127) s_x acc_diag
 *  Output        y = y_off + y_diag + D s_x xq + corr
 * flags: SSDI8_FLAG_FP16_OPERAND selects the paper's FP16 ChunkScan2 operand (above).
 * SSDI8_FLAG_Y_FP16 / SSDI8_FLAG_Y_BF16: `y` points to [B,L,H,P] 16-bit elements; each binary32
 * output value is rounded to nearest even into that format (fp16 overflows to infinity) as it
 * leaves the epilogue, which halves the largest byte stream of the layer.  Not combinable with taps.
 * SSDI8_FLAG_INT8_STATE selects the paper's own inter-chunk state format (Section 4.2, Eq. 4, 7)
 * instead of fp32 states: the chunk-local state goes INT32 -> INT8 in registers and the
 * recurrence is integer with a fixed-point decay, all states sharing the scale s_h[h,p]:
 *   locq = rne(fmul(float(acc_st), fdiv(fmul(s_xs, s_B), s_h)));   Gq = rne(fmul(Gamma_k, 128))
 *   Sq_k = sat(locq + ((Gq * Sq_{k-1} + 64) >> 7)),  Sq_{-1} = rne(fmul(init_state, fdiv(1, s_h)))
 *   hq[k] = Sq_{k-1};  final_state = fmul(float(Sq_{c-1}), s_h);  tap_loc, tap_prev are not written.
 * Bits 8-12
 * select modules (SSDI8_PHASE_*); 0 in those bits runs all five in order.  A partial run
 * reads the intermediates a previous call left in the same workspace (per-module timing,
 * tests); any other bit set gives SSDI8_ERR_UNSUPPORTED.
 * workspace: at least ssdi8_workspace_bytes(dims, flags) bytes, 256-byte aligned; its
 * contents are scratch.  All tensor pointers and the per-channel vectors s_x, s_xs, s_h, corr are
 * 16-byte aligned (SSDI8_ERR_ALIGN otherwise). */
ssdi8_status_t ssdi8_chunk_scan_fwd(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* args,
                                    uint32_t flags, void* workspace, size_t workspace_bytes,
                                    void* stream);

/* The same forward pass for callers that can pass no workspace because they must not, or
 * cannot, allocate device memory: processes whose device-memory budget is fully assigned at
 * start-up, and latency-critical loops that must never reach cudaMalloc / cudaFree (both
 * synchronise the device).  (The paper has no counterpart of this entry point; it exists for
 * deployment only and computes exactly what ssdi8_chunk_scan_fwd computes.)
 *  - The scratch is a fixed array of SSDI8_STATIC_WORKSPACE_BYTES inside the library, held by
 *    every GPU that loads the library until the process exits.  Dimensions that need more
 *    (ssdi8_workspace_bytes(dims, flags) > SSDI8_STATIC_WORKSPACE_BYTES) are rejected with
 *    SSDI8_ERR_WORKSPACE; use ssdi8_chunk_scan_fwd with your own workspace for those.
 *  - The call allocates nothing and frees nothing, on the host or on the device.
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and keeps it for the life of the process; make that first call before any stream
 *    capture begins, and do not reset the device (cudaDeviceReset) afterwards: the kept address
 *    would then be stale.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.
 *    Nothing in it has to start at zero (every region is written before it is read), but two
 *    calls that overlap on the GPU (different streams, no dependency) race on it: order them.
 * Arguments as for ssdi8_chunk_scan_fwd, minus the workspace. */
#define SSDI8_STATIC_WORKSPACE_BYTES (16u << 20)
ssdi8_status_t ssdi8_chunk_scan_fwd_static(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* args,
                                           uint32_t flags, void* stream);

/* The layer step as one call: Eq. 1 quantisation of fp32 x, B, C with the given static step sizes
 * (ssdi8_quantize_act, mode 0) followed by ssdi8_chunk_scan_fwd.  The paper has no counterpart (its
 * modules are separate kernels on device-resident tensors); the arithmetic is exactly that of
 * the two calls it replaces, and so is the result.
 *
 * ssdi8_layer_fwd: every pointer is a DEVICE pointer.  The three quantisers are one launch (x, B and C
 *   must be 16-byte aligned like every other tensor: SSDI8_ERR_ALIGN otherwise, before anything is
 *   enqueued); all kernels run on `stream`, chained by programmatic dependent launch: ChunkCumsum (reads
 *   dt and A only) first, the quantisers' launch beside it, then the state kernel, ChunkBMM beside the
 *   state kernel's last wave, and ChunkScan; no other stream, no event.  The call may be captured into a
 *   CUDA graph.  workspace: 256-byte aligned,
 *   ssdi8_layer_fwd_workspace_bytes(dims, flags) bytes (the int8 tensors plus ssdi8_workspace_bytes).
 * ssdi8_layer_fwd_host: x, B, C, dt, y, final_state, status are HOST pointers (page-locked memory, or
 *   the copies neither overlap nor run asynchronously), the rest DEVICE pointers.  One slice at a
 *   time, a slice being a batch element or, when an element's x exceeds 96 MB, an equal range of its
 *   heads (Algorithm 2 has no term across batch elements or heads): the host->device copies of slice
 *   i+1 and the device->host copy of y of slice i-1 run on two copy streams while the kernels
 *   of slice i run, so both directions of the host link stay busy.  scratch: DEVICE, 256-byte
 *   aligned, ssdi8_layer_fwd_host_scratch_bytes(dims, flags) bytes (two stages of one slice's tensors).
 * Layouts as in ssdi8_fwd_args_t; D, corr, init_state, final_state, status may be NULL.  Both calls
 * return once everything is enqueued and leave `stream` waiting for the last piece of work, so
 * synchronising `stream` completes them.  flags: any of SSDI8_FLAG_INT8_STATE, SSDI8_FLAG_Y_FP16,
 * SSDI8_FLAG_Y_BF16 (`y` then points to 16-bit elements), SSDI8_FLAG_FP16_OPERAND.  The copy streams and
 * events of ssdi8_layer_fwd_host are created at the first call on each device and shared by later calls:
 * calls of ssdi8_layer_fwd_host on one device must not overlap in time.  Errors: as ssdi8_quantize_act / ssdi8_chunk_scan_fwd, plus
 * SSDI8_ERR_WORKSPACE for a short workspace or scratch. */
typedef struct {
  const float* x; const float* B; const float* C; const float* dt;   /* [B,L,H,P], [B,L,G,N] x2, [B,L,H] */
  const float* A; const float* D; const float* corr;                 /* [H], [H], [H*P]                   */
  const float* s_x; const float* s_B; const float* s_C;              /* step sizes of x, B, C             */
  const float* s_xs; const float* s_cb; const float* s_h;            /* internal step sizes               */
  const float* init_state;                                           /* [B,H,P,N]                         */
  float* y; float* final_state; int32_t* status;                     /* [B,L,H,P], [B,H,P,N], 1 word      */
} ssdi8_layer_args_t;
size_t ssdi8_layer_fwd_workspace_bytes(const ssdi8_dims_t* dims, uint32_t flags);
ssdi8_status_t ssdi8_layer_fwd(const ssdi8_dims_t* dims, const ssdi8_layer_args_t* args, void* workspace,
                               size_t workspace_bytes, uint32_t flags, void* stream);
size_t ssdi8_layer_fwd_host_scratch_bytes(const ssdi8_dims_t* dims, uint32_t flags);
ssdi8_status_t ssdi8_layer_fwd_host(const ssdi8_dims_t* dims, const ssdi8_layer_args_t* args, void* scratch,
                                    size_t scratch_bytes, uint32_t flags, void* stream);

/* Static calibration of the internal step sizes (Eq. 1 applied once to the internal
 * tensors of this input; the paper calibrates offline, Section 5 "Quantization Setup"):
 *   s_xs[h,p] = absmax over (b,t) of |fmul(fmul(float(xq), s_x), LUT_state)| / 127
 *   s_cb[g]   = absmax over the causal half of |acc_cb| * fmul(s_C, s_B) / 127
 *   s_h[h,p]  = absmax over init_state and every S_k, all b and n, / 127
 * (each 1 if its absmax is 0).  Reads xq, Bq, Cq, s_x, s_B, s_C, dt, A, init_state of `args`;
 * ignores its other members.  Writes s_xs [H*P], s_cb [G], s_h [H*P]. */
ssdi8_status_t ssdi8_calibrate(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* args,
                               float* s_xs, float* s_cb, float* s_h, void* workspace,
                               size_t workspace_bytes, void* stream);

/* Estimation of the mean-correction vector (Eq. 8): the least-squares optimal per-channel
 * correction of a quantised output is the channel-wise mean of its error, damped by eta (0.15 in
 * the paper's setup):  corr[ch] = eta * mean over r of (y_ref[r][ch] - y_q[r][ch]).
 * y_ref, y_q: [R][Ch] fp32 (for the SSD output R = B*L, Ch = H*P), 16-byte aligned, Ch % 4 == 0.
 * corr: [Ch].  Sums are carried in fp64 in a fixed order (deterministic).  workspace: at least
 * ssdi8_mean_correction_workspace_bytes(Ch) bytes, 16-byte aligned.  The result can be passed as
 * `corr` to ssdi8_chunk_scan_fwd / ssdi8_ssd_step.  (The multi-layer sequential update of
 * Algorithm 1 needs a whole model and is outside this library.) */
size_t ssdi8_mean_correction_workspace_bytes(int64_t Ch);
ssdi8_status_t ssdi8_mean_correction(const float* y_ref, const float* y_q, int64_t R, int64_t Ch,
                                     float eta, float* corr, void* workspace, size_t workspace_bytes,
                                     void* stream);

/* StatePassing alone (Eq. 5-6; Algorithm 2 module 3) on fp32 states.
 *   S_k = fmaf(gamma[b,h,k], S_{k-1}, loc[b,k,h,p,n]),  S_{-1} = init_state or 0
 *   prev[b,k] = S_{k-1} (may be NULL; may alias loc), final_state = S_{c-1} (may be NULL),
 *   hq[b,k] = rne(fmul(S_{k-1}, fdiv(1, s_h[h,p]))) when hq and s_h are non-NULL.
 * loc, prev [B,c,H,P,N]; gamma [B,H,c]; init_state, final_state [B,H,P,N]; hq [B,c,H,P,N]. */
ssdi8_status_t ssdi8_state_passing(const ssdi8_dims_t* dims, const float* loc, const float* gamma,
                                   const float* init_state, float* prev, float* final_state,
                                   int8_t* hq, const float* s_h, void* stream);

/* One recurrent-mode token for every sequence of the batch (the recurrence
 * h_t = exp(dt A) h_{t-1} + dt B_t x_t^T, y_t = C_t h_t + D x_t that the dual form of
 * Algorithm 2 unrolls; the paper gives no algorithm for this mode).  fp32 throughout:
 *   a = exp(dt[b,h] A[h]);  S[p,n] = a S[p,n] + (dt s_x[h,p] s_B[g]) xq[p] Bq[n]
 *   y[p] = s_C[g] sum_n Cq[n] S[p,n] + D[h] s_x[h,p] xq[p] + corr[h,p]   (updated state)
 * xq [B,H,P]; Bq, Cq [B,G,N]; dt [B,H]; state [B,H,P,N] updated IN PLACE; y [B,H,P].
 * dims.seqlen and dims.chunk are ignored.  D and corr may be NULL. */
ssdi8_status_t ssdi8_ssd_step(const ssdi8_dims_t* dims, const int8_t* xq, const float* s_x,
                              const int8_t* Bq, const float* s_B, const int8_t* Cq,
                              const float* s_C, const float* dt, const float* A, const float* D,
                              const float* corr, float* state, float* y, void* stream);

/* dt = softplus(dt_raw + dt_bias[h]) alone (Algorithm 2 module 1, first line), the arithmetic of
 * SSDI8_FLAG_DT_SOFTPLUS: for callers that calibrate step sizes (ssdi8_calibrate takes the positive time
 * step) or run the recurrent step on raw time steps.  dt_raw, dt [rows][H]; dt_bias [H] or NULL; dt may
 * alias dt_raw. */
ssdi8_status_t ssdi8_softplus_dt(const float* dt_raw, const float* dt_bias, int64_t rows, int32_t H, float* dt,
                                 void* stream);

/* Measurement aid (the paper has no counterpart): what tcgen05.mma.kind::i8 sustains on the current
 * device, for the "fraction of the int8 tensor-pipe peak" a benchmark reports.  One CTA per SM issues
 * `mma_per_sm` (rounded down to a multiple of 128, at least 128) dense MMAs of M 128 x N 256 x K 32
 * back to back on operands resident in shared memory, accumulating into tensor memory.  *ops (HOST)
 * receives the number of integer operations the launch performs (2 per multiply-accumulate); divide
 * by the device time of the call, measured by the caller with events on `stream`.  status: 1 word on
 * the DEVICE or NULL, written only if a bounded wait ran out. */
ssdi8_status_t ssdi8_int8_mma_peak(int64_t mma_per_sm, double* ops, int32_t* status, void* stream);

/* Self-test of the time-out path every kernel of this library shares (Section references: none, the
 * paper has no counterpart).  Launches one thread that waits, through the library's bounded mbarrier
 * wait with a cap of 48 polls, on a barrier nothing ever arrives on: no copy is in flight and no
 * tensor memory is held, so nothing can fault or hang.  After about a millisecond the wait gives up,
 * writes SSDI8_ERR_DEVICE_TIMEOUT to *status (DEVICE, 1 word, required) and the kernel returns
 * normally; the context stays usable. */
ssdi8_status_t ssdi8_selftest_bounded_wait(int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SSDI8_H_ */
