// The layer step as one call: Eq. 1 quantisation of fp32 x, B, C with static step sizes and the SSD
// layer forward (Algorithm 2).
// ssdi8_layer_fwd (device buffers): one chain on the caller's stream, linked by programmatic dependent
// launch.  ChunkCumsum reads dt and A only, so the quantisers' launch behind it starts without waiting
// for it and works beside it; the state kernel, ChunkBMM and ChunkScan follow.
// ssdi8_layer_fwd_host (host buffers): the same, one batch element at a time.  Batch elements are
// independent, so the host->device copies of element b+1 and the device->host copy of the
// output of element b-1 run on two copy streams while the kernels of element b run on the
// caller's stream: the PCIe link is busy in both directions for the whole call instead of
// idle during the kernels and one-directional during the copies.  Only stream and event
// plumbing lives here; every arithmetic step is a kernel of this library.
#include <mutex>

#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int kStages = 2;
constexpr uint32_t kLayerFlags = SSDI8_FLAG_FP16_OPERAND | SSDI8_FLAG_INT8_STATE | SSDI8_FLAG_Y_FP16 | SSDI8_FLAG_Y_BF16;

struct StageBuf {
  float *x, *B, *C, *dt, *y, *fin;
  int8_t *xq, *Bq, *Cq;
};
struct Layout {
  StageBuf st[kStages];
  float* dt_full[2];   // dt of a whole batch element (all heads), alternating by element
  void* ws;
  int32_t* status;
  size_t ws_bytes, total;
};

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

Layout make_layout(const ssdi8_dims_t& d1, int full_heads, uint8_t* base, uint32_t flags) {
  Layout lo;
  const size_t nx = (size_t)d1.seqlen * d1.nheads * d1.headdim, nb = (size_t)d1.seqlen * d1.ngroups * d1.dstate;
  const size_t ndt = (size_t)d1.seqlen * d1.nheads, nfin = (size_t)d1.nheads * d1.headdim * d1.dstate;
  size_t o = 0;
  auto take = [&](size_t bytes) { uint8_t* p = base + o; o = up256(o + bytes); return p; };
  for (int s = 0; s < kStages; ++s) {
    lo.st[s].x = reinterpret_cast<float*>(take(nx * 4));
    lo.st[s].B = reinterpret_cast<float*>(take(nb * 4));
    lo.st[s].C = reinterpret_cast<float*>(take(nb * 4));
    lo.st[s].dt = reinterpret_cast<float*>(take(ndt * 4));
    lo.st[s].y = reinterpret_cast<float*>(take(nx * 4));
    lo.st[s].fin = reinterpret_cast<float*>(take(nfin * 4));
    lo.st[s].xq = reinterpret_cast<int8_t*>(take(nx));
    lo.st[s].Bq = reinterpret_cast<int8_t*>(take(nb));
    lo.st[s].Cq = reinterpret_cast<int8_t*>(take(nb));
  }
  for (int e = 0; e < 2; ++e) lo.dt_full[e] = reinterpret_cast<float*>(take((size_t)d1.seqlen * full_heads * 4));
  lo.status = reinterpret_cast<int32_t*>(take(256));
  lo.ws_bytes = ssdi8_workspace_bytes(&d1, flags);
  lo.ws = take(lo.ws_bytes);
  lo.total = o;
  return lo;
}

// copy streams and events of the host-buffer entry point, made once per device and kept for the life of the process
struct Plumbing {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t start = nullptr, in_done[kStages] = {}, cmp_done[kStages] = {}, out_done[kStages] = {};
};
Plumbing g_plumb[64];
std::mutex g_plumb_mu;   // two threads may make their first call on a device at once

ssdi8_status_t get_plumbing(Plumbing** out) {
  int dev = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SSDI8_ERR_CUDA;
  Plumbing& p = g_plumb[dev];
  std::lock_guard<std::mutex> lock(g_plumb_mu);
  if (!p.ready) {
    SSDI8_CUDA_CHECK(cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking));
    SSDI8_CUDA_CHECK(cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking));
    SSDI8_CUDA_CHECK(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
    for (int s = 0; s < kStages; ++s) {
      SSDI8_CUDA_CHECK(cudaEventCreateWithFlags(&p.in_done[s], cudaEventDisableTiming));
      SSDI8_CUDA_CHECK(cudaEventCreateWithFlags(&p.cmp_done[s], cudaEventDisableTiming));
      SSDI8_CUDA_CHECK(cudaEventCreateWithFlags(&p.out_done[s], cudaEventDisableTiming));
    }
    p.ready = true;
  }
  *out = &p;
  return SSDI8_OK;
}

struct LayerWs {
  int8_t *xq, *Bq, *Cq;
  void* ws;
  size_t ws_bytes, total;
};
LayerWs layer_ws(const ssdi8_dims_t& d, uint8_t* base, uint32_t flags) {
  LayerWs w;
  const size_t nx = (size_t)d.batch * d.seqlen * d.nheads * d.headdim;
  const size_t nb = (size_t)d.batch * d.seqlen * d.ngroups * d.dstate;
  size_t o = 0;
  auto take = [&](size_t bytes) { uint8_t* p = base + o; o = up256(o + bytes); return p; };
  w.xq = reinterpret_cast<int8_t*>(take(nx));
  w.Bq = reinterpret_cast<int8_t*>(take(nb));
  w.Cq = reinterpret_cast<int8_t*>(take(nb));
  w.ws_bytes = ssdi8_workspace_bytes(&d, flags);
  w.ws = take(w.ws_bytes);
  w.total = o;
  return w;
}

// quantisers + forward on device tensors, int8 tensors and workspace given; status cleared by the caller
ssdi8_status_t layer_step(const ssdi8_dims_t& d, const ssdi8_layer_args_t& a, const float* x, const float* B,
                          const float* C, const float* dt, const float* init, float* y, float* fin,
                          int32_t* status, int8_t* xq, int8_t* Bq, int8_t* Cq, void* ws, size_t ws_bytes,
                          uint32_t flags, cudaStream_t st) {
  const int64_t T = (int64_t)d.batch * d.seqlen;
  ssdi8_fwd_args_t f = {};
  f.xq = xq; f.Bq = Bq; f.Cq = Cq;
  f.s_x = a.s_x; f.s_B = a.s_B; f.s_C = a.s_C;
  f.dt = dt; f.A = a.A; f.D = a.D; f.corr = a.corr;
  f.s_xs = a.s_xs; f.s_cb = a.s_cb; f.s_h = a.s_h;
  f.init_state = init; f.y = y; f.final_state = fin; f.status = status;
  const uint32_t fl = flags & kLayerFlags;
  ssdi8_status_t s;
  // (the three quantisers are one launch: it needs a power-of-two N, which every supported N is, and 16-byte
  // aligned tensors, which the entry points have checked or provide themselves)
  if ((d.dstate & (d.dstate - 1)) != 0) return SSDI8_ERR_UNSUPPORTED;
  // ChunkCumsum (it reads dt and A only) and the quantisers need nothing of each other.  ChunkCumsum goes
  // first and lets its successor be scheduled once its own wait for the work ahead of the layer is over;
  // the quantisers' launch then starts without a wait and runs beside it, with the wait at the end of its
  // last block (see quant_jobs), so that the state kernel, which waits for the quantisers' launch, has
  // ChunkCumsum complete as well.  One stream, no events.  Measured per step, this chain / ChunkCumsum on a
  // side stream / ChunkCumsum's blocks inside the quantisers' grid: 0.286 / 0.293 / 0.287 ms at batch
  // 8 x 2048 x 80 heads, 0.056 / 0.062 / 0.062 ms at 2048 x 24 heads.
  if ((s = fwd_phases(&d, &f, fl | SSDI8_PHASE_CUMSUM, ws, ws_bytes, st, false)) != SSDI8_OK) return s;
  if ((s = launch_quantize_xbc(x, B, C, T, d.nheads * d.headdim, d.ngroups, d.dstate, a.s_x, a.s_B, a.s_C, xq, Bq, Cq, st,
                               true)) != SSDI8_OK)
    return s;
  // the rest, chained by programmatic dependent launch: the fused state kernel, ChunkBMM (needed by ChunkScan
  // only: launched behind the state kernel, it works beside that kernel's last wave), ChunkScan
  return fwd_phases(&d, &f, fl | SSDI8_PHASE_BMM | SSDI8_PHASE_CHUNK_STATE | SSDI8_PHASE_STATE_PASSING | SSDI8_PHASE_SCAN,
                    ws, ws_bytes, st, false);
}

// How many equal head ranges a batch element is cut into for the host pipeline: halved while a
// slice's fp32 x is larger than 96 MB (below that the fixed cost of a copy outweighs the shorter
// fill and drain of the pipeline: measured on PCIe 5 x16, a 21 MB copy runs at 47 GB/s, a 350 MB
// copy at 55 GB/s), as long as the cut keeps groups whole (and their step-size
// vectors 16-byte aligned) or there is a single group.
int choose_parts(const ssdi8_dims_t& d) {
  int np = 1;
  auto can = [&](int n) {
    if (d.nheads % n != 0) return false;
    if (d.ngroups == 1) return true;
    return d.ngroups % n == 0 && (d.ngroups / n) % 4 == 0;
  };
  const size_t x_bytes = (size_t)d.seqlen * d.nheads * d.headdim * 4;
  while (np < 4 && can(np * 2) && x_bytes / np > ((size_t)96 << 20)) np *= 2;
  return np;
}
ssdi8_dims_t slice_dims(const ssdi8_dims_t& d, int nparts) {
  ssdi8_dims_t s = d;
  s.batch = 1;
  s.nheads = d.nheads / nparts;
  s.ngroups = d.ngroups == 1 ? 1 : d.ngroups / nparts;
  return s;
}

// rows of `width` bytes from one pitched buffer to another; one plain copy when both are compact
cudaError_t copy_rows(void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, size_t rows,
                      cudaMemcpyKind kind, cudaStream_t st) {
  if (dpitch == width && spitch == width) return cudaMemcpyAsync(dst, src, width * rows, kind, st);
  return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, rows, kind, st);
}

bool layer_args_ok(const ssdi8_layer_args_t* a) {
  return a->x && a->B && a->C && a->dt && a->A && a->s_x && a->s_B && a->s_C && a->s_xs && a->s_cb && a->s_h && a->y;
}

}  // namespace
}  // namespace ssdi8

using namespace ssdi8;

extern "C" {

size_t ssdi8_layer_fwd_workspace_bytes(const ssdi8_dims_t* dims, uint32_t flags) {
  if (!dims || dims->batch <= 0 || (flags & ~kLayerFlags)) return 0;
  if (ssdi8_workspace_bytes(dims, flags) == 0) return 0;
  return layer_ws(*dims, nullptr, flags).total;
}

ssdi8_status_t ssdi8_layer_fwd(const ssdi8_dims_t* dims, const ssdi8_layer_args_t* a, void* workspace,
                               size_t workspace_bytes, uint32_t flags, void* stream) {
  if (!dims || !a || !workspace) return SSDI8_ERR_NULL;
  if (!layer_args_ok(a)) return SSDI8_ERR_NULL;
  if (flags & ~kLayerFlags) return SSDI8_ERR_UNSUPPORTED;
  const size_t need = ssdi8_layer_fwd_workspace_bytes(dims, flags);
  if (need == 0) return SSDI8_ERR_SHAPE;
  if (workspace_bytes < need) return SSDI8_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SSDI8_ERR_ALIGN;
  // the quantisers read x, B and C sixteen bytes at a time (the other tensors are checked by the forward pass,
  // also before anything is enqueued)
  if ((reinterpret_cast<uintptr_t>(a->x) | reinterpret_cast<uintptr_t>(a->B) | reinterpret_cast<uintptr_t>(a->C)) & 15)
    return SSDI8_ERR_ALIGN;
  const LayerWs w = layer_ws(*dims, static_cast<uint8_t*>(workspace), flags);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (a->status) SSDI8_CUDA_CHECK(cudaMemsetAsync(a->status, 0, sizeof(int32_t), st));
  return layer_step(*dims, *a, a->x, a->B, a->C, a->dt, a->init_state, a->y, a->final_state, a->status, w.xq, w.Bq,
                    w.Cq, w.ws, w.ws_bytes, flags, st);
}

size_t ssdi8_layer_fwd_host_scratch_bytes(const ssdi8_dims_t* dims, uint32_t flags) {
  if (!dims || dims->batch <= 0) return 0;
  if (ssdi8_workspace_bytes(dims, flags) == 0) return 0;   // unsupported dimensions or flags
  const ssdi8_dims_t d1 = slice_dims(*dims, choose_parts(*dims));
  if (ssdi8_workspace_bytes(&d1, flags) == 0) return 0;
  return make_layout(d1, dims->nheads, nullptr, flags).total;
}

ssdi8_status_t ssdi8_layer_fwd_host(const ssdi8_dims_t* dims, const ssdi8_layer_args_t* a, void* scratch,
                                    size_t scratch_bytes, uint32_t flags, void* stream) {
  if (!dims || !a || !scratch) return SSDI8_ERR_NULL;
  if (!layer_args_ok(a)) return SSDI8_ERR_NULL;
  if (flags & ~kLayerFlags) return SSDI8_ERR_UNSUPPORTED;
  const size_t need = ssdi8_layer_fwd_host_scratch_bytes(dims, flags);
  if (need == 0) return SSDI8_ERR_SHAPE;
  if (scratch_bytes < need) return SSDI8_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(scratch) & 255) return SSDI8_ERR_ALIGN;
  // a slice = one batch element, or an equal part of its heads when an element is large: the
  // pipeline fills and drains with one slice's copies exposed, so smaller slices hide more
  const int nparts = choose_parts(*dims);
  const ssdi8_dims_t d1 = slice_dims(*dims, nparts);
  const Layout lo = make_layout(d1, dims->nheads, static_cast<uint8_t*>(scratch), flags);
  Plumbing* p = nullptr;
  ssdi8_status_t s = get_plumbing(&p);
  if (s != SSDI8_OK) return s;
  cudaStream_t s_cmp = static_cast<cudaStream_t>(stream);
  const size_t L = dims->seqlen, H = dims->nheads, P = dims->headdim, N = dims->dstate, G = dims->ngroups;
  const size_t Hs = d1.nheads, Gs = d1.ngroups;
  const size_t nfin = Hs * P * N;
  const size_t yb = (flags & (SSDI8_FLAG_Y_FP16 | SSDI8_FLAG_Y_BF16)) ? 2 : 4;  // bytes per element of y
  // everything below is ordered after the work already in the caller's stream
  SSDI8_CUDA_CHECK(cudaMemsetAsync(lo.status, 0, sizeof(int32_t), s_cmp));
  SSDI8_CUDA_CHECK(cudaEventRecord(p->start, s_cmp));
  SSDI8_CUDA_CHECK(cudaStreamWaitEvent(p->s_in, p->start, 0));
  SSDI8_CUDA_CHECK(cudaStreamWaitEvent(p->s_out, p->start, 0));

  const int nslices = dims->batch * nparts;
  for (int i = 0; i < nslices; ++i) {
    const size_t b = (size_t)(i / nparts), part = (size_t)(i % nparts);
    const size_t h0 = part * Hs, g0 = (G == 1) ? 0 : part * Gs;   // first head and first group of the slice
    const int st = i % kStages;
    const StageBuf& sb = lo.st[st];
    // inputs of the slice (rows of L tokens, strided in the host tensors, compact on the device):
    // the kernels of slice i - kStages have finished with this stage
    if (i >= kStages) SSDI8_CUDA_CHECK(cudaStreamWaitEvent(p->s_in, p->cmp_done[st], 0));
    SSDI8_CUDA_CHECK(copy_rows(sb.x, Hs * P * 4, a->x + (b * L * H + h0) * P, H * P * 4, Hs * P * 4, L,
                                       cudaMemcpyHostToDevice, p->s_in));
    SSDI8_CUDA_CHECK(copy_rows(sb.B, Gs * N * 4, a->B + (b * L * G + g0) * N, G * N * 4, Gs * N * 4, L,
                                       cudaMemcpyHostToDevice, p->s_in));
    SSDI8_CUDA_CHECK(copy_rows(sb.C, Gs * N * 4, a->C + (b * L * G + g0) * N, G * N * 4, Gs * N * 4, L,
                                       cudaMemcpyHostToDevice, p->s_in));
    // dt has short rows (4 bytes per head): it crosses the link once per element in one piece and is
    // cut into head ranges on the device
    if (nparts == 1) {
      SSDI8_CUDA_CHECK(cudaMemcpyAsync(sb.dt, a->dt + b * L * H, L * H * 4, cudaMemcpyHostToDevice, p->s_in));
    } else {
      if (part == 0)
        SSDI8_CUDA_CHECK(cudaMemcpyAsync(lo.dt_full[b & 1], a->dt + b * L * H, L * H * 4, cudaMemcpyHostToDevice, p->s_in));
      SSDI8_CUDA_CHECK(copy_rows(sb.dt, Hs * 4, lo.dt_full[b & 1] + h0, H * 4, Hs * 4, L, cudaMemcpyDeviceToDevice,
                                 p->s_in));
    }
    SSDI8_CUDA_CHECK(cudaEventRecord(p->in_done[st], p->s_in));
    // kernels of the slice: its inputs have arrived, and y of slice i - kStages has left
    SSDI8_CUDA_CHECK(cudaStreamWaitEvent(s_cmp, p->in_done[st], 0));
    if (i >= kStages) SSDI8_CUDA_CHECK(cudaStreamWaitEvent(s_cmp, p->out_done[st], 0));
    ssdi8_layer_args_t as = *a;   // per-head and per-group vectors of the slice
    as.A = a->A + h0;
    as.D = a->D ? a->D + h0 : nullptr;
    as.corr = a->corr ? a->corr + h0 * P : nullptr;
    as.s_x = a->s_x + h0 * P; as.s_xs = a->s_xs + h0 * P; as.s_h = a->s_h + h0 * P;
    as.s_B = a->s_B + g0; as.s_C = a->s_C + g0; as.s_cb = a->s_cb + g0;
    const size_t fin_off = (b * H + h0) * P * N;
    s = layer_step(d1, as, sb.x, sb.B, sb.C, sb.dt, a->init_state ? a->init_state + fin_off : nullptr, sb.y,
                   a->final_state ? sb.fin : nullptr, lo.status, sb.xq, sb.Bq, sb.Cq, lo.ws, lo.ws_bytes, flags, s_cmp);
    if (s != SSDI8_OK) return s;
    SSDI8_CUDA_CHECK(cudaEventRecord(p->cmp_done[st], s_cmp));
    // outputs of the slice
    SSDI8_CUDA_CHECK(cudaStreamWaitEvent(p->s_out, p->cmp_done[st], 0));
    SSDI8_CUDA_CHECK(copy_rows(reinterpret_cast<uint8_t*>(a->y) + (b * L * H + h0) * P * yb, H * P * yb, sb.y,
                                       Hs * P * yb, Hs * P * yb, L, cudaMemcpyDeviceToHost, p->s_out));
    if (a->final_state)
      SSDI8_CUDA_CHECK(cudaMemcpyAsync(a->final_state + fin_off, sb.fin, nfin * 4, cudaMemcpyDeviceToHost, p->s_out));
    SSDI8_CUDA_CHECK(cudaEventRecord(p->out_done[st], p->s_out));
  }
  // the caller's stream ends after the last copies (the last kStages slices' events cover all)
  for (int st = 0; st < kStages && st < nslices; ++st)
    SSDI8_CUDA_CHECK(cudaStreamWaitEvent(s_cmp, p->out_done[st], 0));
  if (a->status)
    SSDI8_CUDA_CHECK(cudaMemcpyAsync(a->status, lo.status, sizeof(int32_t), cudaMemcpyDeviceToHost, s_cmp));
  return SSDI8_OK;
}

}  // extern "C"
