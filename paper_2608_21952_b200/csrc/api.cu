// C-ABI entry points of libssdi8: argument validation, workspace layout, kernel sequencing.
#include <cstring>
#include <mutex>

#include "kernels.h"

using namespace ssdi8;

namespace {

constexpr uint32_t kFwdFlags = SSDI8_PHASE_ALL | SSDI8_FLAG_FP16_OPERAND | SSDI8_FLAG_INT8_STATE | SSDI8_FLAG_Y_FP16 |
                               SSDI8_FLAG_Y_BF16 | SSDI8_FLAG_DT_SOFTPLUS;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool dims_supported(const ssdi8_dims_t* d, bool need_chunks) {
  if (!d) return false;
  if (d->batch <= 0 || d->nheads <= 0 || d->ngroups <= 0) return false;
  if (d->headdim != 64) return false;
  if (d->dstate != 64 && d->dstate != 128) return false;
  if (d->nheads % d->ngroups != 0) return false;
  if (need_chunks) {
    if (d->chunk != 64 && d->chunk != 128 && d->chunk != 256) return false;
    if (d->seqlen <= 0 || d->seqlen % d->chunk != 0) return false;
  }
  return true;
}

// The kernels are built for sm_100a only (tensor-memory MMA does not exist elsewhere).
// (First use on a device fills the cache under a lock: two threads may make their first call at once.)
ssdi8_status_t check_arch() {
  static int ok_device[64];  // 0 unknown, 1 ok, -1 wrong
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SSDI8_ERR_CUDA;
  if (dev < 0 || dev >= 64) return SSDI8_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (ok_device[dev] == 0) {
    int major = 0, minor = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
      return SSDI8_ERR_CUDA;
    ok_device[dev] = (major == 10 && minor == 0) ? 1 : -1;
  }
  return ok_device[dev] == 1 ? SSDI8_OK : SSDI8_ERR_ARCH;
}

struct Workspace {
  size_t pack, gamma, cbq, loc, hq, total;
};

Workspace layout(const Dims& d, bool fp16_operand = false) {
  Workspace w;
  size_t o = 0;
  const size_t nst = (size_t)d.b * d.c * d.H * d.P * d.N;
  w.pack = o;  o = align_up(o + sizeof(float) * kPackRows * (size_t)d.b * d.H * d.L, 256);
  w.gamma = o; o = align_up(o + sizeof(float) * (size_t)d.b * d.H * d.c, 256);
  w.cbq = o;   o = align_up(o + (size_t)d.b * d.c * d.G * d.Q * d.Q, 256);
  w.loc = o;   o = align_up(o + sizeof(float) * nst, 256);
  w.hq = o;    o = align_up(o + nst, 256);
  (void)fp16_operand;   // the FP16 operand needs no scratch of its own
  w.total = o;
  return w;
}

}  // namespace

extern "C" {

const char* ssdi8_status_string(ssdi8_status_t s) {
  switch (s) {
    case SSDI8_OK: return "ok";
    case SSDI8_ERR_NULL: return "a required pointer is NULL";
    case SSDI8_ERR_SHAPE: return "unsupported or inconsistent dimensions";
    case SSDI8_ERR_ALIGN: return "a pointer is not 16-byte aligned";
    case SSDI8_ERR_WORKSPACE: return "workspace too small";
    case SSDI8_ERR_ARCH: return "device is not compute capability 10.0 (sm_100a)";
    case SSDI8_ERR_CUDA: return "CUDA runtime or launch failure";
    case SSDI8_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case SSDI8_ERR_UNSUPPORTED: return "flag or mode not implemented";
    default: return "unknown status";
  }
}

size_t ssdi8_workspace_bytes(const ssdi8_dims_t* dims, uint32_t flags) {
  if ((flags & ~kFwdFlags) != 0 || !dims_supported(dims, true)) return 0;
  return layout(make_dims(dims), (flags & SSDI8_FLAG_FP16_OPERAND) != 0).total;
}

ssdi8_status_t ssdi8_quantize_act(const float* in, int64_t R, int64_t Ch, int64_t I, float* scale,
                                  int32_t mode, int8_t* out, void* stream) {
  if (!in || !scale) return SSDI8_ERR_NULL;
  if (mode < 0 || mode > 2) return SSDI8_ERR_UNSUPPORTED;
  if (!out && mode != 2) return SSDI8_ERR_NULL;
  if (R < 0 || Ch <= 0 || I <= 0) return SSDI8_ERR_SHAPE;
  if (!(I == 1 || I % 4 == 0) || (Ch * I) % 4 != 0) return SSDI8_ERR_SHAPE;
  if (R * Ch * I >= ((int64_t)1 << 33)) return SSDI8_ERR_SHAPE;
  if (!aligned16(in) || (out && !aligned16(out)) || !aligned16(scale)) return SSDI8_ERR_ALIGN;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_quantize(in, R, Ch, I, scale, mode, out, static_cast<cudaStream_t>(stream));
}

ssdi8_status_t ssdi8_chunk_scan_fwd(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* a,
                                    uint32_t flags, void* workspace, size_t workspace_bytes,
                                    void* stream) {
  return ssdi8::fwd_phases(dims, a, flags, workspace, workspace_bytes, stream, true);
}

}  // extern "C"

namespace ssdi8 {
void workspace_pack_gamma(const Dims& d, void* workspace, float** pack, float** gamma) {
  const Workspace w = layout(d);
  *pack = reinterpret_cast<float*>(static_cast<char*>(workspace) + w.pack);
  *gamma = reinterpret_cast<float*>(static_cast<char*>(workspace) + w.gamma);
}

ssdi8_status_t fwd_phases(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* a, uint32_t flags, void* workspace,
                          size_t workspace_bytes, void* stream, bool clear_status) {
  if (!dims || !a) return SSDI8_ERR_NULL;
  if ((flags & ~kFwdFlags) != 0) return SSDI8_ERR_UNSUPPORTED;
  const bool i8s = (flags & SSDI8_FLAG_INT8_STATE) != 0;
  if ((flags & SSDI8_FLAG_Y_FP16) && (flags & SSDI8_FLAG_Y_BF16)) return SSDI8_ERR_UNSUPPORTED;
  const int ydt = (flags & SSDI8_FLAG_Y_FP16) ? 1 : (flags & SSDI8_FLAG_Y_BF16) ? 2 : 0;
  if (ydt && (a->tap_acc_off || a->tap_rowmax || a->tap_Mq || a->tap_acc_diag)) return SSDI8_ERR_UNSUPPORTED;
  const bool f16op = (flags & SSDI8_FLAG_FP16_OPERAND) != 0;
  if (f16op && (a->tap_acc_off || a->tap_rowmax || a->tap_Mq || a->tap_acc_diag)) return SSDI8_ERR_UNSUPPORTED;
  const uint32_t ph = (flags & SSDI8_PHASE_ALL) ? (flags & SSDI8_PHASE_ALL) : (uint32_t)SSDI8_PHASE_ALL;
  // the INT8 state lives inside the fused ChunkState + StatePassing kernel only
  if (i8s && ((ph & SSDI8_PHASE_CHUNK_STATE) != 0) != ((ph & SSDI8_PHASE_STATE_PASSING) != 0))
    return SSDI8_ERR_UNSUPPORTED;
  if (!dims_supported(dims, true)) return SSDI8_ERR_SHAPE;
  if (!a->xq || !a->Bq || !a->Cq || !a->s_x || !a->s_B || !a->s_C || !a->dt || !a->A || !a->s_xs ||
      !a->s_cb || !a->s_h || !a->y || !workspace)
    return SSDI8_ERR_NULL;
  // the per-channel vectors are read 16 bytes at a time (bulk copies into shared memory, float4 loads)
  const void* ptrs[] = {a->xq, a->Bq, a->Cq, a->dt, a->init_state, a->y, a->final_state,
                        a->s_x, a->s_xs, a->s_h, a->corr,
                        a->tap_cs, a->tap_acc_cb, a->tap_CBq, a->tap_Xsq, a->tap_acc_st, a->tap_loc,
                        a->tap_prev, a->tap_hq, a->tap_acc_off, a->tap_Mq, a->tap_acc_diag};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return SSDI8_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SSDI8_ERR_ALIGN;
  const Dims d = make_dims(dims);
  const Workspace w = layout(d, f16op);
  if (workspace_bytes < w.total) return SSDI8_ERR_WORKSPACE;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  float* pack = reinterpret_cast<float*>(ws + w.pack);
  float* gamma = reinterpret_cast<float*>(ws + w.gamma);
  int8_t* cbq = a->tap_CBq ? a->tap_CBq : reinterpret_cast<int8_t*>(ws + w.cbq);
  float* loc = a->tap_loc ? a->tap_loc : reinterpret_cast<float*>(ws + w.loc);
  int8_t* hq = a->tap_hq ? a->tap_hq : reinterpret_cast<int8_t*>(ws + w.hq);
  if (a->status && clear_status) SSDI8_CUDA_CHECK(cudaMemsetAsync(a->status, 0, sizeof(int32_t), st));

  if ((ph & SSDI8_PHASE_CUMSUM) && (s = launch_cumsum(d, a->dt, a->A, pack, gamma, a->tap_cs, st, a->dt_bias,
                                                     (flags & SSDI8_FLAG_DT_SOFTPLUS) != 0)) != SSDI8_OK)
    return s;
  // ChunkBMM depends on neither ChunkCumsum nor the state kernel and is needed by ChunkScan only.  When the
  // fused state kernel runs in this call, ChunkBMM is launched after it and works beside its last wave.
  const bool fused_state = (ph & SSDI8_PHASE_CHUNK_STATE) && (ph & SSDI8_PHASE_STATE_PASSING);
  const bool bmm_late = (ph & SSDI8_PHASE_BMM) && fused_state;
  if ((ph & SSDI8_PHASE_BMM) && !bmm_late &&
      (s = launch_bmm(d, a->Cq, a->Bq, a->s_C, a->s_B, a->s_cb, cbq, a->tap_acc_cb, nullptr, a->status, st)) !=
          SSDI8_OK)
    return s;
  if ((ph & SSDI8_PHASE_CHUNK_STATE) && (ph & SSDI8_PHASE_STATE_PASSING)) {
    // both modules: the fused chunk-sequential kernel (the fp32 chunk-local states stay on chip)
    if ((s = launch_chunk_state_passing(d, a->xq, a->Bq, a->s_x, a->s_xs, a->s_B, a->s_h, pack, gamma,
                                        a->init_state, hq, a->final_state, a->tap_loc, a->tap_prev,
                                        a->tap_Xsq, a->tap_acc_st, a->status, i8s, st)) != SSDI8_OK)
      return s;
    if (bmm_late && (s = launch_bmm(d, a->Cq, a->Bq, a->s_C, a->s_B, a->s_cb, cbq, a->tap_acc_cb, nullptr, a->status,
                                    st, true)) != SSDI8_OK)
      return s;
  } else {
    if ((ph & SSDI8_PHASE_CHUNK_STATE) &&
        (s = launch_chunk_state(d, a->xq, a->Bq, a->s_x, a->s_xs, a->s_B, pack, loc, a->tap_Xsq,
                                a->tap_acc_st, nullptr, a->status, st)) != SSDI8_OK)
      return s;
    if ((ph & SSDI8_PHASE_STATE_PASSING) &&
        (s = launch_state_passing(d, loc, gamma, a->init_state, a->s_h, a->tap_prev, a->final_state,
                                  hq, nullptr, st)) != SSDI8_OK)
      return s;
  }
  if ((ph & SSDI8_PHASE_SCAN) && f16op)
    return launch_chunk_scan_f16(d, a->xq, a->Cq, cbq, hq, a->s_x, a->s_C, a->s_cb, a->s_h, pack, a->D,
                                 a->corr, a->y, ydt, a->status, st);
  if (ph & SSDI8_PHASE_SCAN) {
    ScanTaps taps = {a->tap_acc_off, a->tap_rowmax, a->tap_Mq, a->tap_acc_diag};
    return launch_chunk_scan(d, a->xq, a->Cq, cbq, hq, a->s_x, a->s_C, a->s_cb, a->s_h, pack,
                             a->D, a->corr, a->y, ydt, a->status, taps, st);
  }
  return SSDI8_OK;
}
}  // namespace ssdi8

extern "C" {

ssdi8_status_t ssdi8_calibrate(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* a, float* s_xs,
                               float* s_cb, float* s_h, void* workspace, size_t workspace_bytes,
                               void* stream) {
  if (!dims || !a) return SSDI8_ERR_NULL;
  if (!dims_supported(dims, true)) return SSDI8_ERR_SHAPE;
  if (!a->xq || !a->Bq || !a->Cq || !a->s_x || !a->s_B || !a->s_C || !a->dt || !a->A || !s_xs ||
      !s_cb || !s_h || !workspace)
    return SSDI8_ERR_NULL;
  const void* ptrs[] = {a->xq, a->Bq, a->Cq, a->dt, a->init_state};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return SSDI8_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SSDI8_ERR_ALIGN;
  const Dims d = make_dims(dims);
  const Workspace w = layout(d);
  if (workspace_bytes < w.total) return SSDI8_ERR_WORKSPACE;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  float* pack = reinterpret_cast<float*>(ws + w.pack);
  float* gamma = reinterpret_cast<float*>(ws + w.gamma);
  float* loc = reinterpret_cast<float*>(ws + w.loc);
  const i64 nhp = (i64)d.H * d.P;
  // the outputs double as the running maxima (bit patterns), finalised in place
  SSDI8_CUDA_CHECK(cudaMemsetAsync(s_xs, 0, sizeof(float) * nhp, st));
  SSDI8_CUDA_CHECK(cudaMemsetAsync(s_cb, 0, sizeof(float) * d.G, st));
  SSDI8_CUDA_CHECK(cudaMemsetAsync(s_h, 0, sizeof(float) * nhp, st));
  if ((s = launch_cumsum(d, a->dt, a->A, pack, gamma, nullptr, st)) != SSDI8_OK) return s;
  if ((s = launch_chunk_state(d, a->xq, a->Bq, a->s_x, nullptr, a->s_B, pack, nullptr, nullptr,
                              nullptr, reinterpret_cast<uint32_t*>(s_xs), nullptr, st)) != SSDI8_OK)
    return s;
  if ((s = launch_finalize_scales(s_xs, nhp, nullptr, nullptr, 0, st)) != SSDI8_OK) return s;
  if ((s = launch_bmm(d, a->Cq, a->Bq, a->s_C, a->s_B, nullptr, nullptr, nullptr,
                      reinterpret_cast<uint32_t*>(s_cb), nullptr, st)) != SSDI8_OK)
    return s;
  if ((s = launch_finalize_scales(s_cb, d.G, a->s_C, a->s_B, 1, st)) != SSDI8_OK) return s;
  if ((s = launch_chunk_state(d, a->xq, a->Bq, a->s_x, s_xs, a->s_B, pack, loc, nullptr,
                              nullptr, nullptr, nullptr, st)) != SSDI8_OK)
    return s;
  if ((s = launch_state_passing(d, loc, gamma, a->init_state, nullptr, nullptr, nullptr, nullptr,
                                reinterpret_cast<uint32_t*>(s_h), st)) != SSDI8_OK)
    return s;
  return launch_finalize_scales(s_h, nhp, nullptr, nullptr, 0, st);
}

ssdi8_status_t ssdi8_state_passing(const ssdi8_dims_t* dims, const float* loc, const float* gamma,
                                   const float* init_state, float* prev, float* final_state,
                                   int8_t* hq, const float* s_h, void* stream) {
  if (!dims || !loc || !gamma) return SSDI8_ERR_NULL;
  if (!dims_supported(dims, true)) return SSDI8_ERR_SHAPE;
  if (hq && !s_h) return SSDI8_ERR_NULL;
  const void* ptrs[] = {loc, init_state, prev, final_state, hq};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return SSDI8_ERR_ALIGN;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_state_passing(make_dims(dims), loc, gamma, init_state, s_h, prev, final_state, hq,
                              nullptr, static_cast<cudaStream_t>(stream));
}

ssdi8_status_t ssdi8_ssd_step(const ssdi8_dims_t* dims, const int8_t* xq, const float* s_x,
                              const int8_t* Bq, const float* s_B, const int8_t* Cq,
                              const float* s_C, const float* dt, const float* A, const float* D,
                              const float* corr, float* state, float* y, void* stream) {
  if (!dims || !xq || !s_x || !Bq || !s_B || !Cq || !s_C || !dt || !A || !state || !y)
    return SSDI8_ERR_NULL;
  if (!dims_supported(dims, false)) return SSDI8_ERR_SHAPE;
  const void* ptrs[] = {xq, Bq, Cq, state, y};
  for (const void* p : ptrs)
    if (!aligned16(p)) return SSDI8_ERR_ALIGN;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_ssd_step(make_dims(dims), xq, s_x, Bq, s_B, Cq, s_C, dt, A, D, corr, state, y,
                         static_cast<cudaStream_t>(stream));
}

ssdi8_status_t ssdi8_quantize_entry(const void* xBC, int32_t dtype, int64_t T, int32_t D, int32_t G, int32_t N,
                                    const float* s_x, const float* s_B, const float* s_C, int8_t* xq,
                                    int8_t* Bq, int8_t* Cq, void* stream) {
  if (!xBC || !s_x || !s_B || !s_C || !xq || !Bq || !Cq) return SSDI8_ERR_NULL;
  if (dtype < 0 || dtype > 2) return SSDI8_ERR_UNSUPPORTED;
  if (T < 0 || D <= 0 || G <= 0 || N <= 0 || D % 4 != 0 || N % 4 != 0) return SSDI8_ERR_SHAPE;
  const void* ptrs[] = {xBC, s_x, xq, Bq, Cq};
  for (const void* p : ptrs)
    if (!aligned16(p)) return SSDI8_ERR_ALIGN;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_quantize_entry(xBC, dtype, T, D, G, N, s_x, s_B, s_C, xq, Bq, Cq, static_cast<cudaStream_t>(stream));
}

size_t ssdi8_mean_correction_workspace_bytes(int64_t Ch) {
  return Ch > 0 ? sizeof(double) * (size_t)kMeanCorrMaxSlabs * (size_t)Ch : 0;
}

ssdi8_status_t ssdi8_mean_correction(const float* y_ref, const float* y_q, int64_t R, int64_t Ch, float eta,
                                     float* corr, void* workspace, size_t workspace_bytes, void* stream) {
  if (!y_ref || !y_q || !corr || !workspace) return SSDI8_ERR_NULL;
  if (R <= 0 || Ch <= 0 || Ch % 4 != 0) return SSDI8_ERR_SHAPE;
  if (!aligned16(y_ref) || !aligned16(y_q) || !aligned16(workspace)) return SSDI8_ERR_ALIGN;
  if (workspace_bytes < ssdi8_mean_correction_workspace_bytes(Ch)) return SSDI8_ERR_WORKSPACE;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_mean_correction(y_ref, y_q, R, Ch, eta, corr, static_cast<double*>(workspace),
                                static_cast<cudaStream_t>(stream));
}

ssdi8_status_t ssdi8_softplus_dt(const float* dt_raw, const float* dt_bias, int64_t rows, int32_t H, float* dt,
                                 void* stream) {
  if (!dt_raw || !dt) return SSDI8_ERR_NULL;
  if (rows < 0 || H <= 0) return SSDI8_ERR_SHAPE;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_softplus_dt(dt_raw, dt_bias, dt, rows, H, static_cast<cudaStream_t>(stream));
}

ssdi8_status_t ssdi8_int8_mma_peak(int64_t mma_per_sm, double* ops, int32_t* status, void* stream) {
  if (!ops) return SSDI8_ERR_NULL;
  const int per_batch = int8_mma_peak_batch();
  if (mma_per_sm < per_batch || mma_per_sm > ((int64_t)1 << 24)) return SSDI8_ERR_SHAPE;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  const int nbatch = (int)(mma_per_sm / per_batch);
  int ctas = 0;
  if ((s = launch_int8_mma_peak(nbatch, status, &ctas, static_cast<cudaStream_t>(stream))) != SSDI8_OK) return s;
  *ops = 2.0 * 128.0 * 256.0 * 32.0 * (double)per_batch * (double)nbatch * (double)ctas;
  return SSDI8_OK;
}

ssdi8_status_t ssdi8_selftest_bounded_wait(int32_t* status, void* stream) {
  if (!status) return SSDI8_ERR_NULL;
  ssdi8_status_t s = check_arch();
  if (s != SSDI8_OK) return s;
  return launch_bounded_wait_expires(status, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------
// Forward pass with library-owned scratch (no allocation by anyone).
//
// Some callers cannot hand the library a workspace: a serving process whose whole device-memory
// budget was carved up at start-up (weights, state caches) has no allocator left to ask, and a
// latency-critical decode/prefill loop must not reach cudaMalloc or cudaFree at all, because both
// synchronise the device.  For them the scratch of the layer forward lives in the array below,
// which every GPU that loads this library holds from load until the process exits.
//
// g_static_ws is a device symbol.  Inside host code its name is only a host-side stand-in, not a
// device address, so the address is looked up once per device with cudaGetSymbolAddress (with
// that device current) and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_ws[SSDI8_STATIC_WORKSPACE_BYTES];

ssdi8_status_t ssdi8_chunk_scan_fwd_static(const ssdi8_dims_t* dims, const ssdi8_fwd_args_t* args,
                                           uint32_t flags, void* stream) {
  if (!dims || !args) return SSDI8_ERR_NULL;
  const size_t need = ssdi8_workspace_bytes(dims, flags);
  if (need == 0)
    return (flags & ~kFwdFlags) ? SSDI8_ERR_UNSUPPORTED : SSDI8_ERR_SHAPE;
  if (need > (size_t)SSDI8_STATIC_WORKSPACE_BYTES) return SSDI8_ERR_WORKSPACE;  // beyond the built-in scratch
  // (before the symbol lookup: on a device of another architecture the lookup itself fails, and the
  // caller should learn that the device is the wrong one)
  const ssdi8_status_t arch = check_arch();
  if (arch != SSDI8_OK) return arch;
  static void* ws_of_device[64];  // resolved address of g_static_ws, per device
  static std::mutex ws_mu;        // two threads may make their first call on a device at once
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SSDI8_ERR_CUDA;
  std::lock_guard<std::mutex> lock(ws_mu);
  if (!ws_of_device[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return SSDI8_ERR_CUDA;
    }
    ws_of_device[dev] = p;
  }
  return ssdi8_chunk_scan_fwd(dims, args, flags, ws_of_device[dev], SSDI8_STATIC_WORKSPACE_BYTES, stream);
}

}  // extern "C"
