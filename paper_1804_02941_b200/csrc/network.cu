// Whole-network inference (Section 5.1: Sketch-A-Net, ResNet-18 and GoogLeNet with all but the first (and last)
// layer binarized): the full-precision layers around the binarized ones as small kernels of their own, and
// dab_network_forward, which queues every layer of a chain on one stream without synchronising.
//
// The glue is not the hot path (the binarized layers are): each kernel is the layer's plain definition, one thread
// per output.  The dense convolution sums its products in fp64 in element order (c, kh, kw), each product and sum
// rounded on its own, and rounds once to fp32, so that its result does not depend on the launch shape.
#include "common.cuh"

namespace dab {

namespace {

constexpr int kGlueThreads = 256;

inline unsigned glue_blocks(int64_t count) {
  int64_t b = (count + kGlueThreads - 1) / kGlueThreads;
  const int64_t cap = (int64_t)sm_count() * 32;
  return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

__global__ void __launch_bounds__(kGlueThreads) conv_dense_kernel(dab_conv_desc d, int Ho, int Wo, const float* __restrict__ x,
                                                                  const float* __restrict__ w, const float* __restrict__ bias,
                                                                  float* __restrict__ y) {
  const int64_t outputs = (int64_t)d.N * d.Cout * Ho * Wo;
  const int n = d.C * d.kh * d.kw;
  for (int64_t oi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; oi < outputs; oi += (int64_t)gridDim.x * blockDim.x) {
    const int wo = (int)(oi % Wo);
    const int ho = (int)((oi / Wo) % Ho);
    const int co = (int)((oi / ((int64_t)Wo * Ho)) % d.Cout);
    const int img = (int)(oi / ((int64_t)Wo * Ho * d.Cout));
    const float* wrow = w + (int64_t)co * n;
    const float* ximg = x + (int64_t)img * d.C * d.H * d.W;
    const int hb = ho * d.stride_h - d.pad_h, wb = wo * d.stride_w - d.pad_w;
    double acc = 0.0;
    for (int c = 0; c < d.C; ++c)
      for (int r = 0; r < d.kh; ++r) {
        const int h = hb + r;
        for (int s = 0; s < d.kw; ++s) {
          const int wq = wb + s;
          double xv = 0.0;
          if ((unsigned)h < (unsigned)d.H && (unsigned)wq < (unsigned)d.W) xv = (double)__ldg(ximg + ((int64_t)c * d.H + h) * d.W + wq);
          acc = __dadd_rn(acc, __dmul_rn(xv, (double)__ldg(wrow + (c * d.kh + r) * d.kw + s)));
        }
      }
    if (bias) acc = __dadd_rn(acc, (double)__ldg(bias + co));
    y[oi] = (float)acc;
  }
}

__global__ void __launch_bounds__(kGlueThreads) affine_kernel(const float* __restrict__ x, int64_t total, int C, int64_t HW,
                                                              const float* __restrict__ scale, const float* __restrict__ shift,
                                                              float* __restrict__ y) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int c = (int)((i / HW) % C);
    y[i] = (float)__dadd_rn(__dmul_rn((double)__ldg(scale + c), (double)x[i]), (double)__ldg(shift + c));
  }
}

__global__ void __launch_bounds__(kGlueThreads) relu_kernel(const float* __restrict__ x, int64_t total, float* __restrict__ y) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = x[i];
    y[i] = v > 0.0f ? v : 0.0f;
  }
}

__global__ void __launch_bounds__(kGlueThreads) add_kernel(const float* __restrict__ a, const float* __restrict__ b, int64_t total,
                                                           float* __restrict__ y) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x)
    y[i] = __fadd_rn(a[i], b[i]);
}

__global__ void __launch_bounds__(kGlueThreads) maxpool_kernel(dab_conv_desc d, int Ho, int Wo, const float* __restrict__ x,
                                                               float* __restrict__ y) {
  const int64_t outputs = (int64_t)d.N * d.C * Ho * Wo;
  for (int64_t oi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; oi < outputs; oi += (int64_t)gridDim.x * blockDim.x) {
    const int wo = (int)(oi % Wo);
    const int ho = (int)((oi / Wo) % Ho);
    const int64_t plane = oi / ((int64_t)Wo * Ho);
    const float* xp = x + plane * d.H * d.W;
    bool seen = false;
    float best = 0.0f;
    for (int r = 0; r < d.kh; ++r)
      for (int s = 0; s < d.kw; ++s) {
        const int h = ho * d.stride_h - d.pad_h + r, wq = wo * d.stride_w - d.pad_w + s;
        if ((unsigned)h < (unsigned)d.H && (unsigned)wq < (unsigned)d.W) {
          const float v = xp[(int64_t)h * d.W + wq];
          if (!seen || v > best) best = v;
          seen = true;
        }
      }
    y[oi] = best;
  }
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
constexpr size_t kAlign = 256;

struct Shape {
  int32_t C, H, W;
  int64_t count(int32_t N) const { return (int64_t)N * C * H * W; }
};

// Geometry of layer `L` applied to a tensor of shape `in`; false if it cannot be applied.
bool layer_desc(const dab_layer& L, int32_t N, const Shape& in, dab_conv_desc* d, Shape* out) {
  d->N = N; d->C = in.C; d->H = in.H; d->W = in.W;
  d->Cout = L.kind == DAB_LAYER_MAXPOOL ? in.C : L.Cout;
  d->kh = L.kh; d->kw = L.kw; d->stride_h = L.stride_h; d->stride_w = L.stride_w; d->pad_h = L.pad_h; d->pad_w = L.pad_w;
  // (the row-length limit of the binarized layers does not apply to pooling and full-precision layers)
  if (d->Cout < 1 || d->kh < 1 || d->kw < 1 || d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0) return false;
  const int64_t eh = (int64_t)d->H + 2 * (int64_t)d->pad_h - d->kh, ew = (int64_t)d->W + 2 * (int64_t)d->pad_w - d->kw;
  if (eh < 0 || ew < 0) return false;
  out->C = d->Cout; out->H = (int32_t)(eh / d->stride_h + 1); out->W = (int32_t)(ew / d->stride_w + 1);
  return true;
}

struct Plan {
  int64_t max_count = 0;   // largest tensor of the chain, elements
  size_t conv_scratch = 0; // largest scratch of a binarized layer
  Shape out{0, 0, 0};
};

// Walks the chain on the host: shapes, argument checks, sizes.  Returns DAB_OK or the status to report.
dab_status plan_network(const dab_layer* layers, int32_t count, int32_t N, Shape in, Plan* plan) {
  if (!layers || count < 1 || N < 1 || in.C < 1 || in.H < 1 || in.W < 1) return DAB_ERR_INVALID_ARG;
  Shape cur = in, saved{0, 0, 0};
  plan->max_count = cur.count(N);
  for (int32_t i = 0; i < count; ++i) {
    const dab_layer& L = layers[i];
    Shape& t = L.on_saved ? saved : cur;
    if (L.on_saved && saved.C == 0) return DAB_ERR_INVALID_ARG;  // nothing was saved
    dab_conv_desc d;
    Shape out = t;
    switch (L.kind) {
      case DAB_LAYER_CONV_DENSE:
        if (!L.d_weights || L.Cout < 1 || !layer_desc(L, N, t, &d, &out)) return DAB_ERR_INVALID_ARG;
        break;
      case DAB_LAYER_CONV_BINARY: {
        if (!L.d_wmask || !L.d_wK || !L.d_walpha || !L.d_wbeta || L.Cout < 1 || L.on_saved) return DAB_ERR_INVALID_ARG;
        if ((int64_t)t.C * L.kh * L.kw > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
        if (!layer_desc(L, N, t, &d, &out)) return DAB_ERR_INVALID_ARG;
        const size_t s = dab_binary_conv_workspace(&d);
        if (s == 0) return DAB_ERR_INVALID_ARG;
        if (s > plan->conv_scratch) plan->conv_scratch = s;
        break;
      }
      case DAB_LAYER_AFFINE:
        if (!L.d_scale || !L.d_shift) return DAB_ERR_INVALID_ARG;
        break;
      case DAB_LAYER_RELU:
        break;
      case DAB_LAYER_MAXPOOL:
        if (!layer_desc(L, N, t, &d, &out)) return DAB_ERR_INVALID_ARG;
        break;
      case DAB_LAYER_SAVE:
        if (L.on_saved) return DAB_ERR_INVALID_ARG;
        saved = cur;
        continue;
      case DAB_LAYER_ADD:
        if (L.on_saved || saved.C != cur.C || saved.H != cur.H || saved.W != cur.W) return DAB_ERR_INVALID_ARG;
        break;
      default:
        return DAB_ERR_INVALID_ARG;
    }
    t = out;
    if (out.count(N) > plan->max_count) plan->max_count = out.count(N);
  }
  plan->out = cur;
  return DAB_OK;
}

}  // namespace
}  // namespace dab

using namespace dab;

extern "C" {

dab_status dab_network_output_shape(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W,
                                    int32_t* Cout, int32_t* Ho, int32_t* Wo) {
  if (!Cout || !Ho || !Wo) return DAB_ERR_INVALID_ARG;
  Plan plan;
  dab_status s = plan_network(layers, count, N, Shape{C, H, W}, &plan);
  if (s != DAB_OK) return s;
  *Cout = plan.out.C; *Ho = plan.out.H; *Wo = plan.out.W;
  return DAB_OK;
}

size_t dab_network_workspace(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W) {
  Plan plan;
  if (plan_network(layers, count, N, Shape{C, H, W}, &plan) != DAB_OK) return 0;
  return 4 * round_up((size_t)plan.max_count * sizeof(float), kAlign) + round_up(plan.conv_scratch, kAlign);
}

dab_status dab_network_forward(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W,
                               const float* d_x, float* d_y, void* d_workspace, size_t workspace_bytes,
                               float* const* h_layer_outputs, void* stream) {
  Plan plan;
  dab_status st = plan_network(layers, count, N, Shape{C, H, W}, &plan);
  if (st != DAB_OK) return st;
  if (!d_x || !d_y) return DAB_ERR_INVALID_ARG;
  const size_t buf = round_up((size_t)plan.max_count * sizeof(float), kAlign);
  if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) || workspace_bytes < 4 * buf + round_up(plan.conv_scratch, kAlign))
    return DAB_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(d_workspace);
  float* pool[4] = {reinterpret_cast<float*>(ws), reinterpret_cast<float*>(ws + buf), reinterpret_cast<float*>(ws + 2 * buf),
                    reinterpret_cast<float*>(ws + 3 * buf)};
  void* scratch = ws + 4 * buf;
  // buffers 0/1 alternate for the running tensor, 2/3 for the remembered one
  const float* cur = d_x;
  const float* saved = nullptr;
  int cur_next = 0, saved_next = 2;
  Shape cs_shape{C, H, W}, sv_shape{0, 0, 0};
  for (int32_t i = 0; i < count; ++i) {
    const dab_layer& L = layers[i];
    float* keep = h_layer_outputs ? h_layer_outputs[i] : nullptr;  // the caller wants this layer's output
    if (L.kind == DAB_LAYER_SAVE) {
      // the remembered tensor is a copy (the running buffers are overwritten two layers on); the running tensor stays
      float* slot = pool[saved_next];
      saved_next = saved_next == 2 ? 3 : 2;
      const size_t bytes = (size_t)cs_shape.count(N) * sizeof(float);
      if (cudaMemcpyAsync(slot, cur, bytes, cudaMemcpyDeviceToDevice, cs) != cudaSuccess) return DAB_ERR_CUDA;
      if (keep && cudaMemcpyAsync(keep, cur, bytes, cudaMemcpyDeviceToDevice, cs) != cudaSuccess) return DAB_ERR_CUDA;
      saved = slot;
      sv_shape = cs_shape;
      continue;
    }
    Shape& shp = L.on_saved ? sv_shape : cs_shape;
    const float* src = L.on_saved ? saved : cur;
    float* dst;
    if (keep) dst = keep;
    else if (L.on_saved) { dst = pool[saved_next]; saved_next = saved_next == 2 ? 3 : 2; }
    else if (i == count - 1) dst = d_y;
    else { dst = pool[cur_next]; cur_next ^= 1; }
    dab_conv_desc d;
    Shape out = shp;
    cudaError_t e = cudaSuccess;
    switch (L.kind) {
      case DAB_LAYER_CONV_DENSE:
        layer_desc(L, N, shp, &d, &out);
        conv_dense_kernel<<<glue_blocks(out.count(N)), kGlueThreads, 0, cs>>>(d, out.H, out.W, src, L.d_weights, L.d_bias, dst);
        e = cudaGetLastError();
        break;
      case DAB_LAYER_CONV_BINARY: {
        layer_desc(L, N, shp, &d, &out);
        dab_status s = dab_binary_conv(&d, src, L.d_wmask, L.ldw, L.d_wK, L.d_walpha, L.d_wbeta, dst, scratch,
                                       round_up(plan.conv_scratch, kAlign), nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr,
                                       stream);
        if (s != DAB_OK) return s;
        break;
      }
      case DAB_LAYER_AFFINE:
        affine_kernel<<<glue_blocks(shp.count(N)), kGlueThreads, 0, cs>>>(src, shp.count(N), shp.C, (int64_t)shp.H * shp.W, L.d_scale,
                                                                          L.d_shift, dst);
        e = cudaGetLastError();
        break;
      case DAB_LAYER_RELU:
        relu_kernel<<<glue_blocks(shp.count(N)), kGlueThreads, 0, cs>>>(src, shp.count(N), dst);
        e = cudaGetLastError();
        break;
      case DAB_LAYER_MAXPOOL:
        layer_desc(L, N, shp, &d, &out);
        maxpool_kernel<<<glue_blocks(out.count(N)), kGlueThreads, 0, cs>>>(d, out.H, out.W, src, dst);
        e = cudaGetLastError();
        break;
      case DAB_LAYER_ADD:
        add_kernel<<<glue_blocks(shp.count(N)), kGlueThreads, 0, cs>>>(cur, saved, shp.count(N), dst);
        e = cudaGetLastError();
        break;
      default:
        return DAB_ERR_INVALID_ARG;
    }
    if (e != cudaSuccess) return DAB_ERR_CUDA;
    shp = out;
    if (L.on_saved) saved = dst;
    else cur = dst;
  }
  if (cur != d_y &&
      cudaMemcpyAsync(d_y, cur, (size_t)cs_shape.count(N) * sizeof(float), cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
    return DAB_ERR_CUDA;
  return DAB_OK;
}

}  // extern "C"
