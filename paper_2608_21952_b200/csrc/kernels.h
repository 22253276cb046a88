// Host-side launchers of the SSDi8 kernels (internal to the library).
#pragma once
#include "common.cuh"

#include <utility>

namespace ssdi8 {

// kernel<<<grid, block, smem, st>>>(args...) with programmatic stream serialization allowed: the
// kernel may be scheduled while its predecessor in the stream drains (see pdl_wait in common.cuh)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

ssdi8_status_t launch_quantize(const float* in, i64 R, i64 Ch, i64 I, float* scale, int mode,
                               int8_t* out, cudaStream_t st);

// the layer's three static quantisers as one launch: x [T][D] with D step sizes, B and C [T][G N] with G
// step sizes each (N a power of two, D and N multiples of 4).
// after_cumsum: the launch directly follows launch_cumsum of the same layer in the same stream and runs beside
// it (see quant_jobs).
ssdi8_status_t launch_quantize_xbc(const float* x, const float* B, const float* C, i64 T_, int D, int G, int N,
                                   const float* s_x, const float* s_B, const float* s_C, int8_t* xq, int8_t* Bq,
                                   int8_t* Cq, cudaStream_t st, bool after_cumsum = false);

// Per-(batch, head, chunk) pack of kPackRows rows of Q floats: cs, dt, woff, atok, wmax, lut (see
// cumsum.cu); element (u, row, i) at pack[(u * kPackRows + row) * Q + i], u = (b*H + h)*c + k.
constexpr int kPackRows = 6;
enum { PACK_CS = 0, PACK_DT = 1, PACK_WOFF = 2, PACK_ATOK = 3, PACK_WMAX = 4, PACK_LUT = 5 };

// xBC [T][D + 2 G N] (dtype 0 fp32, 1 fp16, 2 bf16) -> xq [T][D], Bq, Cq [T][G N], static step sizes
ssdi8_status_t launch_quantize_entry(const void* xBC, int dtype, i64 T_, int D, int G, int N, const float* s_x,
                                     const float* s_B, const float* s_C, int8_t* xq, int8_t* Bq, int8_t* Cq,
                                     cudaStream_t st);

// ssdi8_chunk_scan_fwd's body; clear_status = false leaves the status word alone (callers that run
// the modules as several calls clear it once themselves)
ssdi8_status_t fwd_phases(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* a, uint32_t flags, void* workspace,
                          size_t workspace_bytes, void* stream, bool clear_status);

// where ChunkCumsum's outputs live inside a workspace of ssdi8_workspace_bytes
void workspace_pack_gamma(const Dims& d, void* workspace, float** pack, float** gamma);

// pack [b,H,c,6,Q], gamma [b,H,c], tap_cs [b,H,c,Q] or NULL
// softplus: dt is the raw time step, dt = softplus(dt + dt_bias[h]) is applied first (dt_bias may be NULL)
ssdi8_status_t launch_cumsum(const Dims& d, const float* dt, const float* A, float* pack,
                             float* gamma, float* tap_cs, cudaStream_t st, const float* dt_bias = nullptr,
                             bool softplus = false);
ssdi8_status_t launch_softplus_dt(const float* dt_raw, const float* dt_bias, float* out, i64 rows, int H,
                                  cudaStream_t st);

// acc_cb (tap, may be NULL), CBq (may be NULL when s_cb is NULL), absmax_acc: per-group
// running max of |acc_cb| over the causal half (calibration; may be NULL).  after_state_kernel: the launch
// directly follows launch_chunk_state_passing in the same stream and may run beside it (see bmm.cu)
ssdi8_status_t launch_bmm(const Dims& d, const int8_t* Cq, const int8_t* Bq, const float* s_C,
                          const float* s_B, const float* s_cb, int8_t* CBq, int32_t* tap_acc,
                          uint32_t* absmax_acc, int32_t* status, cudaStream_t st, bool after_state_kernel = false);

// absmax_xs: per-channel running max (as binary32 bits) of |x_scaled| (calibration; may be
// NULL).  When absmax_xs is non-NULL only that is computed.
ssdi8_status_t launch_chunk_state(const Dims& d, const int8_t* xq, const int8_t* Bq,
                                  const float* s_x, const float* s_xs, const float* s_B,
                                  const float* pack, float* loc, int8_t* tap_Xsq,
                                  int32_t* tap_acc, uint32_t* absmax_xs, int32_t* status,
                                  cudaStream_t st);

// ChunkState and StatePassing in one chunk-sequential kernel (loc never leaves the chip)
ssdi8_status_t launch_chunk_state_passing(const Dims& d, const int8_t* xq, const int8_t* Bq,
                                          const float* s_x, const float* s_xs, const float* s_B,
                                          const float* s_h, const float* pack, const float* gamma,
                                          const float* init, int8_t* hq, float* final_state,
                                          float* tap_loc, float* tap_prev, int8_t* tap_Xsq,
                                          int32_t* tap_acc, int32_t* status, bool int8_state,
                                          cudaStream_t st);

// absmax_h: per-channel running max (binary32 bits) of |S| over init, prev and final
ssdi8_status_t launch_state_passing(const Dims& d, const float* loc, const float* gamma,
                                    const float* init, const float* s_h, float* prev,
                                    float* final_state, int8_t* hq, uint32_t* absmax_h,
                                    cudaStream_t st);

struct ScanTaps {
  int32_t* acc_off; float* rowmax; int8_t* Mq; int32_t* acc_diag;
};

// the same with the paper's FP16 ChunkScan2 operand
ssdi8_status_t launch_chunk_scan_f16(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                     const int8_t* CBq, const int8_t* hq, const float* s_x, const float* s_C,
                                     const float* s_cb, const float* s_h, const float* pack, const float* D,
                                     const float* corr, void* y, int ydt, int32_t* status, cudaStream_t st);

ssdi8_status_t launch_chunk_scan(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                 const int8_t* CBq, const int8_t* hq, const float* s_x,
                                 const float* s_C, const float* s_cb, const float* s_h,
                                 const float* pack, const float* D,
                                 const float* corr, void* y, int ydt, int32_t* status,
                                 const ScanTaps& taps, cudaStream_t st);

ssdi8_status_t launch_ssd_step(const Dims& d, const int8_t* xq, const float* s_x,
                               const int8_t* Bq, const float* s_B, const int8_t* Cq,
                               const float* s_C, const float* dt, const float* A, const float* D,
                               const float* corr, float* state, float* y, cudaStream_t st);

// Eq. 8: corr[ch] = eta * mean_r (y[r][ch] - yq[r][ch]); partial holds kMeanCorrMaxSlabs * Ch doubles
constexpr int kMeanCorrMaxSlabs = 256;
int mean_correction_slabs(i64 R);
ssdi8_status_t launch_mean_correction(const float* y, const float* yq, i64 R, i64 Ch, float eta, float* corr,
                                      double* partial, cudaStream_t st);

// measurement aid and self-test (selftest.cu): `nbatch` batches of int8_mma_peak_batch() MMAs of
// M 128 x N 256 x K 32 on every SM (ctas = number of CTAs launched); a bounded wait that runs out
ssdi8_status_t launch_int8_mma_peak(int nbatch, int32_t* status, int* ctas, cudaStream_t st);
int int8_mma_peak_batch();
ssdi8_status_t launch_bounded_wait_expires(int32_t* status, cudaStream_t st);

// scale[k] = bits[k] == 0 ? 1 : fdiv(as_float(bits[k]) [* mul], 127)   (in place)
ssdi8_status_t launch_finalize_scales(float* scale_bits, i64 n, const float* mul_a,
                                      const float* mul_b, int bits_are_int, cudaStream_t st);

}  // namespace ssdi8
