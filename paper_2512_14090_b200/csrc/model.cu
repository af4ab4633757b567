// Host side of the library: status plumbing, the model object (folded weights + the
// L x {4,8,16,32} bank of packed weights), the evaluation plan that shares work between
// candidate schemes, aiq_forward / aiq_eval_schemes, and the analytic arithmetic intensity.
#include "common.cuh"

#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <tuple>
#include <vector>

namespace aiq {

// ---------------------------------------------------------------------------------------
// status plumbing
// ---------------------------------------------------------------------------------------
static thread_local char t_err[512] = "";
static thread_local int64_t t_launches = 0, t_layer_evals = 0, t_layer_evals_unshared = 0;
// process-wide knobs (aiq_set_eval_options / aiq_set_compute_path): atomics, so a thread that
// changes them while another evaluates gives that call either the old or the new value
static std::atomic<int> g_opt_chunk{0};
static std::atomic<int> g_opt_share{1};
static std::atomic<int> g_opt_path{AIQ_PATH_AUTO};
static std::atomic<int> g_opt_per_tensor{0};  // scale granularity of models created afterwards
static std::atomic<int> g_opt_fuse{5};        // bit 0: basic blocks as one kernel; inverted-residual blocks as one kernel:
                                              // bit 1: wherever eligible, bit 2: where measured faster (mb_block_pays)
static std::atomic<int> g_opt_fuse_pool{1};
static std::atomic<int> g_opt_small_pass{1024};   // image-schemes per pass below which the small view runs   // average pool inside the last convolution's epilogue

aiq_status_t set_error(aiq_status_t status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(t_err, sizeof(t_err), fmt, ap);
  va_end(ap);
  return status;
}

void count_launch() { ++t_launches; }

// ---- per-kernel event timing ---------------------------------------------------------
struct ProfiledLaunch { int kind; cudaEvent_t start, stop; };
static thread_local bool t_profiling = false;
static thread_local std::vector<ProfiledLaunch>* t_prof = nullptr;     // launches of this session
static thread_local std::vector<cudaEvent_t>* t_event_pool = nullptr;  // reusable events
static thread_local aiq_kernel_profile_t t_work[AIQ_KERNEL_KINDS];

static cudaEvent_t take_event() {
  if (t_event_pool && !t_event_pool->empty()) {
    cudaEvent_t e = t_event_pool->back();
    t_event_pool->pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}

LaunchScope::LaunchScope(int kind, cudaStream_t stream, double flops, double bytes) : slot_(-1), stream_(stream) {
  if (!t_profiling || kind < 0 || kind >= AIQ_KERNEL_KINDS) return;
  ProfiledLaunch pl = {kind, take_event(), take_event()};
  if (!pl.start || !pl.stop) return;
  t_work[kind].launches += 1;
  t_work[kind].flops += flops;
  t_work[kind].bytes += bytes;
  cudaEventRecord(pl.start, stream);
  t_prof->push_back(pl);
  slot_ = (int)t_prof->size() - 1;
}

LaunchScope::~LaunchScope() {
  if (slot_ >= 0) cudaEventRecord((*t_prof)[slot_].stop, stream_);
}

aiq_status_t check_device_sm100() {
  static int cached[64];   // 0 unknown, 1 ok, 2 not sm_100
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_error(AIQ_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev >= 0 && dev < 64 && cached[dev]) {
    if (cached[dev] == 1) return AIQ_OK;
    return set_error(AIQ_ERR_NOT_SM100, "device %d is not compute capability 10.x", dev);
  }
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return set_error(AIQ_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
  if (dev >= 0 && dev < 64) cached[dev] = (major == 10) ? 1 : 2;
  if (major != 10) return set_error(AIQ_ERR_NOT_SM100, "device %d is compute capability %d.x, need 10.x", dev, major);
  return AIQ_OK;
}

aiq_status_t current_device_props(DeviceProps* out) {
  static std::atomic<int> ready[64];
  static DeviceProps cache[64];
  int dev = 0;
  AIQ_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && ready[dev].load(std::memory_order_acquire)) { *out = cache[dev]; return AIQ_OK; }
  DeviceProps p = {dev, 0, 0};
  AIQ_CUDA_TRY(cudaDeviceGetAttribute(&p.n_sms, cudaDevAttrMultiProcessorCount, dev));
  AIQ_CUDA_TRY(cudaDeviceGetAttribute(&p.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  if (dev >= 0 && dev < 64) { cache[dev] = p; ready[dev].store(1, std::memory_order_release); }
  *out = p;
  return AIQ_OK;
}

static const int kBitsList[4] = {4, 8, 16, 32};
static inline int bits_index(int bits) { return bits == 4 ? 0 : bits == 8 ? 1 : bits == 16 ? 2 : bits == 32 ? 3 : -1; }

}  // namespace aiq

// ---------------------------------------------------------------------------------------
// model object
// ---------------------------------------------------------------------------------------
struct LayerInfo {
  aiq_layer_desc_t d;
  int K, Hi, Wi, Ho, Wo;
  size_t out_bytes;        // per image, split format (fc: float32 logits)
  float* Wf;
  float* bias;
  uint8_t* packed[4];
  float* scales[4];
  int slot;                // activation slot of the output (-1: fc)
  // layers of an inverted-residual block the fused kernel can take (see mb_block.cu): operand images of the
  // 1x1 layers per 4- / 8-bit version, coefficient rows (expansion: 4 / 8 bits; depthwise: every bit-width),
  // hidden channels per chunk the images were built for (0: none built)
  uint8_t* mb_tile[2];
  float* mb_coef[4];
  int mb_nh;
};

struct aiq_model {
  std::vector<LayerInfo> layers;
  int in_c, in_h, in_w;
  std::vector<int> order;            // execution order (every layer after its operands)
  std::vector<size_t> slot_bytes;    // per-image capacity of each activation slot
  void* dev_mem;
  size_t dev_bytes;
  int act_format;                    // ACT_F32, ACT_SPLIT or ACT_RS (see common.cuh)
  int32_t* status_word;              // device word raised by a kernel whose bounded wait expired
  std::vector<int> block_tail;       // per layer: the second convolution of the basic block this layer opens
                                     // (the pair can run as one kernel), or -1
  int pool_layer;                    // the layer whose epilogue can do the classifier's average pool, or -1
  aiq_model* small_view = nullptr;   // the same weights with split activations and the pixel-tile kernels, for passes
                                     // too small to fill the row-streaming kernels (owned; else nullptr)
  std::vector<int> mb_mid, mb_tail;  // per layer: the depthwise and the projection layer of the inverted-residual
                                     // block this (expansion) layer opens (the three can run as one kernel), or -1
};

namespace aiq {

static aiq_status_t infer_shapes(const aiq_arch_desc_t* arch, std::vector<LayerInfo>& L, std::vector<int>& order) {
  if (!arch || !arch->layers || arch->n_layers <= 0 || arch->in_c <= 0 || arch->in_h <= 0 || arch->in_w <= 0)
    return set_error(AIQ_ERR_INVALID_ARG, "architecture description is empty");
  const int n = arch->n_layers;
  L.assign(n, LayerInfo());
  for (int i = 0; i < n; ++i) {
    L[i].d = arch->layers[i];
    const aiq_layer_desc_t& d = L[i].d;
    if (d.kind < AIQ_LAYER_CONV || d.kind > AIQ_LAYER_FC) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: kind %d", i, d.kind);
    if (d.act < AIQ_ACT_NONE || d.act > AIQ_ACT_RELU6) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: act %d", i, d.act);
    if (d.input < -1 || d.input >= n || d.input == i) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: input %d", i, d.input);
    if (d.residual < -1 || d.residual >= n || d.residual == i) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: residual %d", i, d.residual);
    if (d.cin <= 0 || d.cout <= 0) return set_error(AIQ_ERR_SHAPE, "layer %d: cin %d cout %d", i, d.cin, d.cout);
    if (d.kind == AIQ_LAYER_FC) {
      if (i != n - 1) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: the classifier must be the last layer", i);
      if (d.input < 0 || d.residual >= 0) return set_error(AIQ_ERR_INVALID_ARG, "layer %d: classifier wiring", i);
    } else {
      if (d.ksize < 1 || d.ksize > 7 || d.stride < 1 || d.stride > 4 || d.pad < 0 || d.pad > 3)
        return set_error(AIQ_ERR_SHAPE, "layer %d: ksize %d stride %d pad %d", i, d.ksize, d.stride, d.pad);
      if (d.kind == AIQ_LAYER_DEPTHWISE && (d.ksize != 3 || d.pad != 1 || d.cin != d.cout || (d.cout & 3) || d.input < 0))
        return set_error(AIQ_ERR_SHAPE, "layer %d: depthwise must be 3x3, pad 1, cin == cout, channels a multiple of 4", i);
    }
  }
  if (L[n - 1].d.kind != AIQ_LAYER_FC) return set_error(AIQ_ERR_INVALID_ARG, "the last layer must be a classifier (fc)");

  // execution order: depth-first over operands; a cycle shows up as a revisit of an open node
  order.clear();
  std::vector<int> state(n, 0);
  struct Frame { int layer, stage; };
  for (int root = 0; root < n; ++root) {
    if (state[root]) continue;
    std::vector<Frame> st;
    st.push_back({root, 0});
    state[root] = 1;
    while (!st.empty()) {
      Frame& f = st.back();
      const int dep = f.stage == 0 ? L[f.layer].d.input : f.stage == 1 ? L[f.layer].d.residual : -2;
      if (dep == -2) {
        state[f.layer] = 2;
        order.push_back(f.layer);
        st.pop_back();
        continue;
      }
      ++f.stage;
      if (dep < 0 || state[dep] == 2) continue;
      if (state[dep] == 1) return set_error(AIQ_ERR_INVALID_ARG, "wiring has a cycle through layer %d", dep);
      state[dep] = 1;
      st.push_back({dep, 0});
    }
  }

  for (int i : order) {
    LayerInfo& li = L[i];
    const aiq_layer_desc_t& d = li.d;
    int cin_avail, hi, wi;
    if (d.input < 0) { cin_avail = arch->in_c; hi = arch->in_h; wi = arch->in_w; }
    else {
      if (L[d.input].d.kind == AIQ_LAYER_FC) return set_error(AIQ_ERR_INVALID_ARG, "layer %d reads the classifier", i);
      cin_avail = L[d.input].d.cout; hi = L[d.input].Ho; wi = L[d.input].Wo;
    }
    if (cin_avail != d.cin) return set_error(AIQ_ERR_SHAPE, "layer %d: cin %d but its input has %d channels", i, d.cin, cin_avail);
    li.Hi = hi; li.Wi = wi;
    if (d.kind == AIQ_LAYER_FC) {
      li.K = d.cin; li.Hi = 1; li.Wi = 1; li.Ho = 1; li.Wo = 1; li.out_bytes = (size_t)d.cout * 4;   // reads the pooled vector
      continue;
    }
    li.Ho = (hi + 2 * d.pad - d.ksize) / d.stride + 1;
    li.Wo = (wi + 2 * d.pad - d.ksize) / d.stride + 1;
    if (li.Ho <= 0 || li.Wo <= 0) return set_error(AIQ_ERR_SHAPE, "layer %d: empty output", i);
    li.K = (d.kind == AIQ_LAYER_DEPTHWISE ? 1 : d.cin) * d.ksize * d.ksize;
    li.out_bytes = split_image_bytes(li.Ho, li.Wo, d.cout);
    if (d.residual >= 0) {
      const LayerInfo& r = L[d.residual];
      if (r.d.kind == AIQ_LAYER_FC || r.d.cout != d.cout || r.Ho != li.Ho || r.Wo != li.Wo)
        return set_error(AIQ_ERR_SHAPE, "layer %d: residual from layer %d has another shape", i, d.residual);
    }
  }
  return AIQ_OK;
}

static ConvGeom make_geom(const aiq_model* m, const LayerInfo& li, int B) {
  ConvGeom g = {};
  g.B = B; g.H = li.Hi; g.W = li.Wi; g.Cin = li.d.cin; g.Ho = li.Ho; g.Wo = li.Wo; g.Cout = li.d.cout;
  g.ks = li.d.ksize; g.stride = li.d.stride; g.pad = li.d.pad; g.act = li.d.act; g.K = li.K;
  g.Cs_in = padded_channels(li.d.cin); g.Cs_out = padded_channels(li.d.cout);
  g.in_is_nchw = li.d.input < 0 ? 1 : 0;          // the network input is float32 NCHW
  g.act_format = m->act_format;
  return g;
}

// 0: float32 kernels only; 1: small-channel 3x3 / 1x1 tensor-core kernel; 2: pointwise tensor-core
// kernel; 3: row-streaming tensor-core kernel (models stored in ACT_RS)
static int layer_tensor_kind(const aiq_model* m, const LayerInfo& li) {
  if (li.d.kind != AIQ_LAYER_CONV) return 0;
  const ConvGeom g = make_geom(m, li, 1);
  if (conv_rs_eligible(g)) return 3;
  if (conv_tc_eligible(g)) return 1;
  if (conv_pw_tc_eligible(g)) return 2;
  return 0;
}
static bool layer_on_tensor_cores(const aiq_model* m, const LayerInfo& li) { return layer_tensor_kind(m, li) != 0; }

static void assign_slots(aiq_model* m) {
  const int n = (int)m->layers.size();
  std::vector<int> pos(n), last_use(n, -1);
  for (int i = 0; i < n; ++i) pos[m->order[i]] = i;
  for (int l = 0; l < n; ++l) {
    const aiq_layer_desc_t& d = m->layers[l].d;
    if (d.input >= 0) last_use[d.input] = std::max(last_use[d.input], pos[l]);
    if (d.residual >= 0) last_use[d.residual] = std::max(last_use[d.residual], pos[l]);
  }
  std::vector<int> owner;   // layer currently held by each slot, -1 = free
  m->slot_bytes.clear();
  for (int i = 0; i < n; ++i) {
    const int l = m->order[i];
    LayerInfo& li = m->layers[l];
    if (li.d.kind == AIQ_LAYER_FC) { li.slot = -1; }
    else {
      int s = -1;
      for (size_t k = 0; k < owner.size(); ++k) if (owner[k] < 0) { s = (int)k; break; }
      if (s < 0) { s = (int)owner.size(); owner.push_back(-1); m->slot_bytes.push_back(0); }
      owner[s] = l;
      li.slot = s;
      m->slot_bytes[s] = std::max(m->slot_bytes[s], li.out_bytes);
    }
    for (size_t k = 0; k < owner.size(); ++k)
      if (owner[k] >= 0 && last_use[owner[k]] <= i && owner[k] != l) owner[k] = -1;
    if (li.slot >= 0 && last_use[l] < 0) owner[li.slot] = -1;   // never consumed
  }
}

// Inverted-residual blocks by structure alone: an expansion 1x1 (no shortcut) that feeds only a depthwise 3x3
// that feeds only a projection 1x1 whose shortcut (if any) is the expansion's input.  mid / tail: per
// expansion layer the depthwise and the projection layer, else -1.
static void find_mb_structure(const std::vector<LayerInfo>& L, std::vector<int>& mid, std::vector<int>& tail) {
  const int n = (int)L.size();
  mid.assign(n, -1);
  tail.assign(n, -1);
  std::vector<int> uses(n, 0);
  for (const LayerInfo& li : L) {
    if (li.d.input >= 0) uses[li.d.input]++;
    if (li.d.residual >= 0) uses[li.d.residual]++;
  }
  for (int le = 0; le < n; ++le) {
    const LayerInfo& e = L[le];
    if (e.d.kind != AIQ_LAYER_CONV || e.d.ksize != 1 || e.d.input < 0 || e.d.residual >= 0 || uses[le] != 1) continue;
    if (e.d.cin % 8 != 0 || e.d.cout % 16 != 0) continue;
    for (int ld = 0; ld < n; ++ld) {
      const LayerInfo& d = L[ld];
      if (d.d.kind != AIQ_LAYER_DEPTHWISE || d.d.ksize != 3 || d.d.input != le || d.d.residual >= 0 || uses[ld] != 1) continue;
      for (int lp = 0; lp < n; ++lp) {
        const LayerInfo& pr = L[lp];
        if (pr.d.kind != AIQ_LAYER_CONV || pr.d.ksize != 1 || pr.d.input != ld) continue;
        if (pr.d.residual >= 0 && pr.d.residual != e.d.input) continue;
        mid[le] = ld;
        tail[le] = lp;
      }
    }
  }
}

struct ModelLayout {
  size_t total, staging_off, flag_off;
  std::vector<size_t> wf, bias;
  std::vector<size_t> packed[4], scales[4];
  std::vector<size_t> mb_tile[2], mb_coef[4];       // 0: the layer has none
};

static ModelLayout model_layout(const std::vector<LayerInfo>& L) {
  ModelLayout lay;
  size_t off = 0, staging = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  lay.flag_off = take(256);
  for (const LayerInfo& li : L) {
    const size_t n = li.d.cout, k = li.K;
    lay.wf.push_back(take(n * k * 4));
    lay.bias.push_back(take(n * 4));
    for (int b = 0; b < 4; ++b) {
      lay.packed[b].push_back(take(n * row_bytes((int)k, kBitsList[b])));
      lay.scales[b].push_back(take(n * 4));
    }
    staging = std::max(staging, align_up(n * k * 4, 256) + 5 * align_up(n * 4, 256));
  }
  lay.staging_off = take(staging);
  // operand images of inverted-residual blocks, sized for either chunk width the kernel may choose
  for (int b = 0; b < 2; ++b) lay.mb_tile[b].assign(L.size(), 0);
  for (int b = 0; b < 4; ++b) lay.mb_coef[b].assign(L.size(), 0);
  std::vector<int> mid, tail;
  find_mb_structure(L, mid, tail);
  for (size_t le = 0; le < L.size(); ++le) {
    if (tail[le] < 0) continue;
    const int ld = mid[le], lp = tail[le];
    const int ch = L[le].d.cout, cs_in = padded_channels(L[le].d.cin), cs_out = padded_channels(L[lp].d.cout);
    size_t et = 0, pt = 0, ec = 0, dc = 0;
    for (int nh = 32; nh <= 64; nh *= 2) {
      const size_t chunks = (size_t)(ch + nh - 1) / nh;
      et = std::max(et, chunks * mb_etile_bytes(cs_in, nh));
      pt = std::max(pt, chunks * mb_ptile_bytes(cs_out, nh));
      ec = std::max(ec, chunks * 2 * nh * 4);
      dc = std::max(dc, chunks * 11 * nh * 4);
    }
    for (int b = 0; b < 2; ++b) {
      lay.mb_tile[b][le] = take(et);
      lay.mb_coef[b][le] = take(ec);
      lay.mb_tile[b][lp] = take(pt);
    }
    for (int b = 0; b < 4; ++b) lay.mb_coef[b][ld] = take(dc);
  }
  lay.total = off;
  return lay;
}

// Everything about a model that depends on the activation format: the format itself (from the requested
// compute path and what the layers allow), per-image tensor sizes, the fused blocks and pooled epilogue the
// format's kernels can take, and the activation slots.
static void derive_format(aiq_model* m, int opt_path) {
  for (LayerInfo& li : m->layers)
    if (li.d.kind != AIQ_LAYER_FC) li.out_bytes = split_image_bytes(li.Ho, li.Wo, li.d.cout);
  // Row-streaming storage when every layer can live in it: a 3x3 stem on the network input, then
  // only dense convolutions the row-streaming kernel takes, then the classifier.
  m->act_format = ACT_RS;
  bool all_rs = opt_path == AIQ_PATH_AUTO || opt_path == AIQ_PATH_TENSOR;
  for (const LayerInfo& li : m->layers) {
    if (!all_rs || li.d.kind == AIQ_LAYER_FC) continue;
    if (li.d.input < 0)
      all_rs = li.d.kind == AIQ_LAYER_CONV && li.d.ksize == 3 && li.d.pad == 1 && li.d.cin <= 4 && li.d.stride <= 2 &&
               (li.d.cout == 16 || li.d.cout == 32 || li.d.cout == 64) && li.Wo % 8 == 0 && li.Wo <= 64;
    else
      all_rs = layer_tensor_kind(m, li) == 3;
  }
  if (!all_rs) {
    m->act_format = ACT_SPLIT;                    // tentatively, to ask which layers would qualify
    bool any_tc = false;
    for (const LayerInfo& li : m->layers) any_tc = any_tc || layer_on_tensor_cores(m, li);
    m->act_format = (opt_path == AIQ_PATH_TENSOR || opt_path == AIQ_PATH_TENSOR_TILES || (opt_path == AIQ_PATH_AUTO && any_tc))
                        ? ACT_SPLIT : ACT_F32;
  }
  if (m->act_format == ACT_RS)
    for (LayerInfo& li : m->layers)
      if (li.d.kind != AIQ_LAYER_FC) li.out_bytes = rs_image_bytes(li.Ho, li.Wo, li.d.cout);
  // identity-shortcut basic blocks that the fused block kernel takes: conv1 (3x3, ReLU) feeds only conv2
  // (3x3, ReLU) and conv2 adds conv1's input
  m->block_tail.assign(m->layers.size(), -1);
  m->pool_layer = -1;
  if (m->act_format == ACT_RS) {
    const int n = (int)m->layers.size();
    std::vector<int> uses(n, 0);
    for (const LayerInfo& li : m->layers) {
      if (li.d.input >= 0) uses[li.d.input]++;
      if (li.d.residual >= 0) uses[li.d.residual]++;
    }
    // the classifier's input: pooled inside its producer's epilogue when nothing else reads that tensor
    const int last = m->layers.back().d.input;
    if (uses[last] == 1 && m->layers[last].d.input >= 0 && layer_tensor_kind(m, m->layers[last]) == 3 &&
        conv_rs_pool_fusable(make_geom(m, m->layers[last], 1)))
      m->pool_layer = last;
    for (int l1 = 0; l1 < n; ++l1) {
      const LayerInfo& a = m->layers[l1];
      if (a.d.kind != AIQ_LAYER_CONV || a.d.input < 0 || a.d.residual >= 0 || a.d.act != AIQ_ACT_RELU || uses[l1] != 1) continue;
      for (int l2 = 0; l2 < n; ++l2) {
        const LayerInfo& b = m->layers[l2];
        if (b.d.kind == AIQ_LAYER_CONV && b.d.input == l1 && b.d.residual == a.d.input && b.d.act == AIQ_ACT_RELU &&
            conv_rs_block_eligible(make_geom(m, a, 1)) && conv_rs_block_eligible(make_geom(m, b, 1)) && a.d.cin == b.d.cin)
          m->block_tail[l1] = l2;
      }
    }
  }
  // inverted-residual blocks that the fused block kernel takes (structure: find_mb_structure; shape and
  // memory: mb_block_chunk_channels, on split activations with both 1x1 layers on the tensor cores)
  m->mb_mid.assign(m->layers.size(), -1);
  m->mb_tail.assign(m->layers.size(), -1);
  for (LayerInfo& li : m->layers) li.mb_nh = 0;
  if (m->act_format == ACT_SPLIT) {
    std::vector<int> mid, tail;
    find_mb_structure(m->layers, mid, tail);
    for (size_t le = 0; le < m->layers.size(); ++le) {
      if (tail[le] < 0) continue;
      LayerInfo& e = m->layers[le];
      LayerInfo& d = m->layers[mid[le]];
      LayerInfo& pr = m->layers[tail[le]];
      if (!layer_on_tensor_cores(m, e) || !layer_on_tensor_cores(m, pr)) continue;
      const int nh = mb_block_chunk_channels(make_geom(m, e, 1), make_geom(m, d, 1), make_geom(m, pr, 1));
      if (!nh) continue;
      m->mb_mid[le] = mid[le];
      m->mb_tail[le] = tail[le];
      e.mb_nh = d.mb_nh = pr.mb_nh = nh;
    }
  }
  assign_slots(m);
}

}  // namespace aiq

extern "C" size_t aiq_model_bytes(const aiq_arch_desc_t* arch) {
  std::vector<LayerInfo> L;
  std::vector<int> order;
  if (aiq::infer_shapes(arch, L, order) != AIQ_OK) return 0;
  return aiq::model_layout(L).total;
}

extern "C" aiq_status_t aiq_model_create(const aiq_arch_desc_t* arch, const aiq_layer_weights_t* weights,
                                         void* dev_mem, size_t dev_bytes, void* stream_, aiq_model_t** out) {
  using namespace aiq;
  if (out) *out = nullptr;
  if (!arch || !weights || !dev_mem || !out) return set_error(AIQ_ERR_INVALID_ARG, "aiq_model_create: null pointer");
  if (((uintptr_t)dev_mem) & 255) return set_error(AIQ_ERR_INVALID_ARG, "aiq_model_create: dev_mem not 256-byte aligned");
  aiq_model* m = new (std::nothrow) aiq_model();
  if (!m) return set_error(AIQ_ERR_INVALID_ARG, "out of host memory");
  aiq_status_t st = infer_shapes(arch, m->layers, m->order);
  if (st != AIQ_OK) { delete m; return st; }
  for (int i = 0; i < arch->n_layers; ++i) {
    const aiq_layer_weights_t& w = weights[i];
    if (!w.W || (m->layers[i].d.has_bn && (!w.gamma || !w.beta || !w.mean || !w.var))) {
      delete m;
      return set_error(AIQ_ERR_INVALID_ARG, "layer %d: missing weight pointers", i);
    }
  }
  const ModelLayout lay = model_layout(m->layers);
  if (dev_bytes < lay.total) {
    delete m;
    return set_error(AIQ_ERR_WORKSPACE_TOO_SMALL, "model needs %zu device bytes, got %zu", lay.total, dev_bytes);
  }
  st = check_device_sm100();
  if (st != AIQ_OK) { delete m; return st; }
  m->in_c = arch->in_c; m->in_h = arch->in_h; m->in_w = arch->in_w;
  m->dev_mem = dev_mem; m->dev_bytes = dev_bytes;
  derive_format(m, g_opt_path.load());
  cudaStream_t stream = (cudaStream_t)stream_;
  uint8_t* base = static_cast<uint8_t*>(dev_mem);
  int32_t* flag = reinterpret_cast<int32_t*>(base + lay.flag_off);
  m->status_word = flag + 1;                      // zeroed with the flag region below

  auto fail = [&](aiq_status_t s) { delete m; return s; };
#define CREATE_TRY(expr)                                                                    \
  do {                                                                                      \
    cudaError_t e__ = (expr);                                                               \
    if (e__ != cudaSuccess)                                                                 \
      return fail(set_error(AIQ_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)));       \
  } while (0)

  const bool per_tensor = g_opt_per_tensor.load() != 0;
  CREATE_TRY(cudaMemsetAsync(flag, 0, 256, stream));
  for (size_t i = 0; i < m->layers.size(); ++i) {
    LayerInfo& li = m->layers[i];
    const size_t n = li.d.cout, k = li.K;
    li.Wf = reinterpret_cast<float*>(base + lay.wf[i]);
    li.bias = reinterpret_cast<float*>(base + lay.bias[i]);
    for (int b = 0; b < 4; ++b) {
      li.packed[b] = base + lay.packed[b][i];
      li.scales[b] = reinterpret_cast<float*>(base + lay.scales[b][i]);
    }
    const aiq_layer_weights_t& w = weights[i];
    if (li.d.has_bn) {
      float* sW = reinterpret_cast<float*>(base + lay.staging_off);
      const size_t vec = align_up(n * 4, 256);
      uint8_t* sv = base + lay.staging_off + align_up(n * k * 4, 256);
      float* sG = reinterpret_cast<float*>(sv);
      float* sB = reinterpret_cast<float*>(sv + vec);
      float* sM = reinterpret_cast<float*>(sv + 2 * vec);
      float* sV = reinterpret_cast<float*>(sv + 3 * vec);
      CREATE_TRY(cudaMemcpyAsync(sW, w.W, n * k * 4, cudaMemcpyHostToDevice, stream));
      CREATE_TRY(cudaMemcpyAsync(sG, w.gamma, n * 4, cudaMemcpyHostToDevice, stream));
      CREATE_TRY(cudaMemcpyAsync(sB, w.beta, n * 4, cudaMemcpyHostToDevice, stream));
      CREATE_TRY(cudaMemcpyAsync(sM, w.mean, n * 4, cudaMemcpyHostToDevice, stream));
      CREATE_TRY(cudaMemcpyAsync(sV, w.var, n * 4, cudaMemcpyHostToDevice, stream));
      st = launch_fold_bn(sW, sG, sB, sM, sV, (int)n, (int)k, 1e-5f, li.Wf, li.bias, stream);
      if (st != AIQ_OK) return fail(st);
    } else {
      CREATE_TRY(cudaMemcpyAsync(li.Wf, w.W, n * k * 4, cudaMemcpyHostToDevice, stream));
      if (w.bias) CREATE_TRY(cudaMemcpyAsync(li.bias, w.bias, n * 4, cudaMemcpyHostToDevice, stream));
      else CREATE_TRY(cudaMemsetAsync(li.bias, 0, n * 4, stream));
    }
    {
      void* packed4[4] = {li.packed[0], li.packed[1], li.packed[2], li.packed[3]};
      st = launch_quantize_bank(li.Wf, (int)n, (int)k, packed4, li.scales, flag,
                                per_tensor ? reinterpret_cast<uint32_t*>(flag + 2) : nullptr, stream);
      if (st != AIQ_OK) return fail(st);
    }
  }
  // operand images of the fused inverted-residual blocks, from the packed codes just written
  for (size_t le = 0; le < m->layers.size(); ++le) {
    if (m->mb_tail[le] < 0) continue;
    const int ld = m->mb_mid[le], lp = m->mb_tail[le];
    LayerInfo& e = m->layers[le];
    LayerInfo& d = m->layers[ld];
    LayerInfo& pr = m->layers[lp];
    const int nh = e.mb_nh;
    for (int b = 0; b < 2; ++b) {
      e.mb_tile[b] = base + lay.mb_tile[b][le];
      e.mb_coef[b] = reinterpret_cast<float*>(base + lay.mb_coef[b][le]);
      pr.mb_tile[b] = base + lay.mb_tile[b][lp];
      st = launch_mb_build_tiles(0, e.packed[b], e.scales[b], e.bias, kBitsList[b], e.d.cout, e.K, nh,
                                 padded_channels(e.d.cin), e.mb_tile[b], e.mb_coef[b], stream);
      if (st != AIQ_OK) return fail(st);
      st = launch_mb_build_tiles(1, pr.packed[b], pr.scales[b], pr.bias, kBitsList[b], pr.d.cout, pr.K, nh,
                                 padded_channels(pr.d.cout), pr.mb_tile[b], nullptr, stream);
      if (st != AIQ_OK) return fail(st);
    }
    for (int b = 0; b < 4; ++b) {
      d.mb_coef[b] = reinterpret_cast<float*>(base + lay.mb_coef[b][ld]);
      st = launch_mb_build_tiles(2, d.packed[b], d.scales[b], d.bias, kBitsList[b], d.d.cout, d.K, nh, 0, nullptr,
                                 d.mb_coef[b], stream);
      if (st != AIQ_OK) return fail(st);
    }
  }
  int32_t host_flag = 0;
  CREATE_TRY(cudaMemcpyAsync(&host_flag, flag, 4, cudaMemcpyDeviceToHost, stream));
  CREATE_TRY(cudaStreamSynchronize(stream));
#undef CREATE_TRY
  if (host_flag == 2) return fail(set_error(AIQ_ERR_TIMEOUT, "a bounded wait inside the quantizer expired"));
  if (host_flag) return fail(set_error(AIQ_ERR_NONFINITE, "a weight is NaN or infinite"));
  // Row-streaming kernels take a group of 8 or 16 images as their unit of work; a pass of a few hundred images
  // leaves most SMs idle.  Under the automatic path the model also keeps the pixel-tile view of the same weights.
  if (m->act_format == ACT_RS && g_opt_path.load() == AIQ_PATH_AUTO) {
    aiq_model* v = new (std::nothrow) aiq_model(*m);
    if (v) {
      v->small_view = nullptr;
      derive_format(v, AIQ_PATH_TENSOR_TILES);
      m->small_view = v;
    }
  }
  *out = m;
  return AIQ_OK;
}

extern "C" void aiq_model_destroy(aiq_model_t* model) {
  if (model) delete model->small_view;
  delete model;
}
extern "C" aiq_status_t aiq_model_status(const aiq_model_t* model, void* stream_) {
  using namespace aiq;
  if (!model) return set_error(AIQ_ERR_INVALID_ARG, "aiq_model_status: null model");
  cudaStream_t stream = (cudaStream_t)stream_;
  int32_t dev_status = 0;
  AIQ_CUDA_TRY(cudaMemcpyAsync(&dev_status, model->status_word, 4, cudaMemcpyDeviceToHost, stream));
  AIQ_CUDA_TRY(cudaStreamSynchronize(stream));
  if (dev_status) {
    AIQ_CUDA_TRY(cudaMemsetAsync(model->status_word, 0, 4, stream));
    return set_error(AIQ_ERR_TIMEOUT, "a bounded wait inside a kernel expired; outputs of that call are invalid");
  }
  return AIQ_OK;
}

extern "C" aiq_status_t aiq_debug_expire_wait(const aiq_model_t* model, int64_t limit_cycles, void* stream_) {
  using namespace aiq;
  if (!model) return set_error(AIQ_ERR_INVALID_ARG, "aiq_debug_expire_wait: null model");
  if (limit_cycles <= 0 || limit_cycles > 2000000000ll)
    return set_error(AIQ_ERR_INVALID_ARG, "aiq_debug_expire_wait: limit_cycles=%lld outside (0, 2e9]", (long long)limit_cycles);
  aiq_status_t st = check_device_sm100();
  if (st != AIQ_OK) return st;
  return launch_expire_wait(model->status_word, limit_cycles, nullptr, (cudaStream_t)stream_);
}

extern "C" int aiq_model_num_layers(const aiq_model_t* model) { return model ? (int)model->layers.size() : -1; }
extern "C" int aiq_model_num_classes(const aiq_model_t* model) { return model ? model->layers.back().d.cout : -1; }

extern "C" aiq_status_t aiq_model_layer_folded(const aiq_model_t* model, int layer, const float** Wf,
                                               const float** bias, int* N, int* K) {
  if (!model || layer < 0 || layer >= (int)model->layers.size())
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_model_layer_folded: layer %d", layer);
  const LayerInfo& li = model->layers[layer];
  if (Wf) *Wf = li.Wf;
  if (bias) *bias = li.bias;
  if (N) *N = li.d.cout;
  if (K) *K = li.K;
  return AIQ_OK;
}

extern "C" aiq_status_t aiq_model_layer_packed(const aiq_model_t* model, int layer, int bits,
                                               const void** packed, const float** scales) {
  if (!model || layer < 0 || layer >= (int)model->layers.size())
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_model_layer_packed: layer %d", layer);
  const int bi = aiq::bits_index(bits);
  if (bi < 0) return aiq::set_error(AIQ_ERR_UNSUPPORTED_BITS, "aiq_model_layer_packed: bits=%d", bits);
  if (packed) *packed = model->layers[layer].packed[bi];
  if (scales) *scales = model->layers[layer].scales[bi];
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// evaluation plan
// ---------------------------------------------------------------------------------------
namespace aiq {

// Workspace layout for a chunk of B images and up to S schemes:
//   [ job records | counts | pooled S*B*C | logits S*B*classes | slot 0 | slot 1 | ... ]
struct WsLayout {
  size_t jobs_off, jobs_bytes, counts_off, pooled_off, logits_off, total;
  std::vector<size_t> slot_off;
};

static size_t jobs_capacity(const aiq_model* m, int S) {
  // every layer: up to S jobs; the head adds pool + argmax records
  return ((size_t)m->layers.size() + 2) * (size_t)S;
}

static WsLayout ws_layout(const aiq_model* m, int B, int S) {
  WsLayout w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.jobs_bytes = jobs_capacity(m, S) * sizeof(LayerJob);
  w.jobs_off = take(w.jobs_bytes);
  w.counts_off = take((size_t)S * 4);
  const LayerInfo& fc = m->layers.back();
  w.pooled_off = take((size_t)S * B * fc.d.cin * 4);
  w.logits_off = take((size_t)S * B * fc.d.cout * 4);
  const size_t Bslot = m->act_format == ACT_RS ? (size_t)rs_padded_batch(B) : (size_t)B;   // images a version occupies
  for (size_t e : m->slot_bytes) w.slot_off.push_back(take((size_t)S * Bslot * e));
  w.total = off;
  return w;
}

struct alignas(64) TensorMapBytes { uint8_t b[128]; };   // storage of one CUtensorMap

struct LayerPlan {
  int n_versions = 0;
  int n_tc = 0;                         // leading jobs that run on the tensor-core kernel (4- / 8-bit weights)
  int n_tc16 = 0, n_tc32 = 0;           // then those with 16-bit and with 32-bit weights (tc_kind 1 only)
  int tc_kind = 0;                      // which tensor-core kernel (see layer_tensor_kind)
  bool pools = false;                   // its jobs write the classifier's pooled input instead of the tensor
  bool skipped = false;                 // first convolution of a fused block: evaluated inside its partner's kernel
  int fused_head = -1;                  // last layer of a fused block: the first layer it absorbs
  int fused_mid = -1;                   // inverted-residual block: the depthwise layer between the two (else -1)
  double weight_bytes = 0.0;            // packed weights + scales + biases over all jobs
  double weight_bytes_tc = 0.0, weight_bytes_tc16 = 0.0, weight_bytes_tc32 = 0.0;
  TensorMapBytes maps[2];               // [0] over the input slot (tensor-core layers); [1] over the output slot
                                        // (pointwise layers) or the second input map (row-streaming layers)
  size_t job_first = 0;                 // index of the first job record of this layer
  // fc only
  int n_pool = 0;
  size_t pool_first = 0, argmax_first = 0;
  std::vector<std::pair<int, int>> bit_groups;   // (first job, count) per bit-width for qlinear
  std::vector<int> group_bits;
};

struct EvalPlan {
  int batch_capacity = 0;               // images the plan's buffers are laid out for
  std::vector<LayerPlan> lp;            // per layer
  std::vector<LayerJob> jobs;           // host image of all job records
  std::vector<int> final_version;       // per scheme: version of the classifier output
  int n_final = 0;
  int64_t versions_total = 0;
};

// Builds the job records for `S` schemes over a chunk of B images.  With sharing on, a
// (layer, version) is keyed by (bit-width, version of its input, version of its residual):
// candidates that agree on a prefix of the network reuse its activations.
static aiq_status_t build_plan(const aiq_model* m, const uint8_t* schemes, int S, int B, bool share,
                               uint8_t* ws, const WsLayout& wl, float* user_logits, EvalPlan& plan) {
  const int n = (int)m->layers.size();
  for (int s = 0; s < S; ++s)
    for (int l = 0; l < n; ++l)
      if (!bits_ok(schemes[(size_t)s * n + l]))
        return set_error(AIQ_ERR_UNSUPPORTED_BITS, "scheme %d, layer %d: bits=%d", s, l, (int)schemes[(size_t)s * n + l]);
  plan.lp.assign(n, LayerPlan());
  plan.jobs.clear();
  plan.batch_capacity = B;
  std::vector<std::vector<int>> ver(n, std::vector<int>(S, 0));   // ver[l][s]
  std::vector<std::vector<std::tuple<int, int, int>>> all_keys(n);   // per layer and version: (bits, input version, residual version)
  const bool fuse = (g_opt_fuse.load() & 1) != 0;
  const bool fuse_mb_all = (g_opt_fuse.load() & 2) != 0, fuse_mb_auto = (g_opt_fuse.load() & 4) != 0;
  // a basic block runs as one kernel when every scheme gives both of its convolutions 4 or 8 bits
  std::vector<int> fuse_head(n, -1);
  if (fuse)
    for (int l1 = 0; l1 < n; ++l1) {
      const int l2 = m->block_tail[l1];
      if (l2 < 0) continue;
      bool ok = true;
      for (int s = 0; s < S && ok; ++s) ok = schemes[(size_t)s * n + l1] <= 8 && schemes[(size_t)s * n + l2] <= 8;
      if (ok) fuse_head[l2] = l1;
    }
  // an inverted-residual block runs as one kernel when every scheme gives its two 1x1 layers 4 or 8 bits
  std::vector<int> mb_head(n, -1);
  std::vector<char> mb_absorbed(n, 0);
  if (fuse_mb_all || fuse_mb_auto)
    for (int le = 0; le < n; ++le) {
      const int lt = m->mb_tail[le];
      if (lt < 0) continue;
      bool ok = true;
      for (int s = 0; s < S && ok; ++s) ok = schemes[(size_t)s * n + le] <= 8 && schemes[(size_t)s * n + lt] <= 8;
      if (ok && !fuse_mb_all)
        ok = mb_block_pays(make_geom(m, m->layers[m->mb_mid[le]], B), make_geom(m, m->layers[lt], B));
      if (ok) { mb_head[lt] = le; mb_absorbed[le] = 1; mb_absorbed[m->mb_mid[le]] = 1; }
    }
  float* const pooled_base = reinterpret_cast<float*>(ws + wl.pooled_off);
  auto slot_ptr = [&](int layer, int version) -> uint8_t* {
    const LayerInfo& li = m->layers[layer];
    const size_t Bslot = m->act_format == ACT_RS ? (size_t)rs_padded_batch(B) : (size_t)B;
    return ws + wl.slot_off[li.slot] + (size_t)version * Bslot * li.out_bytes;
  };
  for (int l : m->order) {
    const LayerInfo& li = m->layers[l];
    LayerPlan& lp = plan.lp[l];
    std::map<std::tuple<int, int, int>, int> seen;
    std::vector<std::tuple<int, int, int>> keys;   // per version
    for (int s = 0; s < S; ++s) {
      const int bits = schemes[(size_t)s * n + l];
      const int vin = li.d.input >= 0 ? ver[li.d.input][s] : 0;
      const int vres = li.d.residual >= 0 ? ver[li.d.residual][s] : 0;
      if (share) {
        auto key = std::make_tuple(bits, vin, vres);
        auto it = seen.find(key);
        if (it == seen.end()) {
          it = seen.emplace(key, (int)keys.size()).first;
          keys.push_back(key);
        }
        ver[l][s] = it->second;
      } else {
        ver[l][s] = s;
        keys.push_back(std::make_tuple(bits, vin, vres));
      }
    }
    lp.n_versions = (int)keys.size();
    plan.versions_total += lp.n_versions;
    all_keys[l] = keys;
    if (li.d.kind != AIQ_LAYER_FC && m->block_tail[l] >= 0 && fuse_head[m->block_tail[l]] == l) {
      lp.skipped = true;                   // evaluated inside the kernel of the block's second convolution
      continue;
    }
    if (li.d.kind != AIQ_LAYER_FC && mb_absorbed[l]) {
      lp.skipped = true;                   // evaluated inside the kernel of the block's projection layer
      continue;
    }
    if (li.d.kind != AIQ_LAYER_FC && mb_head[l] >= 0) {
      // fused inverted-residual block: one job per version of the projection, carrying the weights of the
      // expansion and depthwise versions it descends from
      const int le = mb_head[l], ld = m->mb_mid[le];
      const LayerInfo& ex = m->layers[le];
      const LayerInfo& dw = m->layers[ld];
      lp.fused_head = le;
      lp.fused_mid = ld;
      lp.job_first = plan.jobs.size();
      plan.versions_total += 2 * lp.n_versions - plan.lp[le].n_versions - plan.lp[ld].n_versions;
      for (int v = 0; v < lp.n_versions; ++v) {
        const int bits = std::get<0>(keys[v]);
        const std::tuple<int, int, int>& kd = all_keys[ld][std::get<1>(keys[v])];
        const std::tuple<int, int, int>& ke = all_keys[le][std::get<1>(kd)];
        const int bits_d = std::get<0>(kd), bits_e = std::get<0>(ke), vin = std::get<1>(ke);
        LayerJob j = {};
        j.in = slot_ptr(ex.d.input, vin);
        j.res = li.d.residual >= 0 ? slot_ptr(li.d.residual, std::get<2>(keys[v])) : nullptr;
        j.out = slot_ptr(l, v);
        j.in_version = vin;
        j.out_version = v;
        j.w = li.mb_tile[bits_index(bits)];                  // operand images (see LayerJob)
        j.scale = li.scales[bits_index(bits)];
        j.bias = li.bias;
        j.bits = bits;
        j.w_pre = ex.mb_tile[bits_index(bits_e)];
        j.scale_pre = ex.mb_coef[bits_index(bits_e)];
        j.bits_pre = bits_e;
        j.scale_mid = dw.mb_coef[bits_index(bits_d)];
        j.bits_mid = bits_d;
        plan.jobs.push_back(j);
        lp.n_tc++;
        lp.weight_bytes_tc += (double)li.d.cout * (row_bytes(li.K, bits) + 8.0) + (double)ex.d.cout * (row_bytes(ex.K, bits_e) + 8.0) +
                              (double)dw.d.cout * (row_bytes(dw.K, bits_d) + 8.0);
      }
      continue;
    }
    if (li.d.kind != AIQ_LAYER_FC && fuse_head[l] >= 0) {
      // fused block: one job per version of this (second) convolution, carrying the first one's weights
      const int l1 = fuse_head[l];
      const LayerInfo& head = m->layers[l1];
      const LayerInfo& src = m->layers[head.d.input];
      lp.fused_head = l1;
      lp.job_first = plan.jobs.size();
      aiq_status_t st = conv_rs_encode_maps(make_geom(m, head, B), ws + wl.slot_off[src.slot], B,
                                            plan.lp[head.d.input].n_versions, &lp.maps[0]);
      if (st != AIQ_OK) return st;
      plan.versions_total += lp.n_versions - plan.lp[l1].n_versions;   // conv1 runs once per job of the block
      for (int v = 0; v < lp.n_versions; ++v) {
        const int bits = std::get<0>(keys[v]);
        const std::tuple<int, int, int>& k1 = all_keys[l1][std::get<1>(keys[v])];
        const int bits1 = std::get<0>(k1), vin = std::get<1>(k1);
        LayerJob j = {};
        j.in = slot_ptr(head.d.input, vin);
        j.res = j.in;
        j.out = slot_ptr(l, v);
        j.in_version = vin;
        j.out_version = v;
        j.w = li.packed[bits_index(bits)];
        j.scale = li.scales[bits_index(bits)];
        j.bias = li.bias;
        j.bits = bits;
        j.w_pre = head.packed[bits_index(bits1)];
        j.scale_pre = head.scales[bits_index(bits1)];
        j.bias_pre = head.bias;
        j.bits_pre = bits1;
        plan.jobs.push_back(j);
        lp.n_tc++;
        lp.weight_bytes_tc += (double)li.d.cout * (row_bytes(li.K, bits) + 8.0) + (double)head.d.cout * (row_bytes(head.K, bits1) + 8.0);
      }
      continue;
    }
    if (li.d.kind != AIQ_LAYER_FC) {
      lp.job_first = plan.jobs.size();
      // job order: versions the tensor-core kernel takes first, grouped by weight class
      // (4- / 8-bit codes, then 16-bit, then 32-bit where the kernel can hold their pieces)
      const bool tc_layer = layer_on_tensor_cores(m, li);
      const int tkind = layer_tensor_kind(m, li);
      const bool tc_wide = tc_layer;            // every tensor-core kernel also takes 16- / 32-bit weights (two pieces)
      const ConvGeom g_cls = make_geom(m, li, B);
      auto job_class = [&](int bits) -> int {      // 0: codes, 1: 16-bit, 2: 32-bit on tensor cores; 3: float32 kernel
        if (tc_layer && bits <= 8) return 0;
        if (tc_wide && bits == 16 && (tkind != 1 || conv_tc_bits_ok(g_cls, 16))) return 1;
        if (tc_wide && bits == 32 && (tkind != 1 || conv_tc_bits_ok(g_cls, 32))) return 2;
        return 3;
      };
      std::vector<int> vorder;
      for (int pass = 0; pass < 4; ++pass)
        for (int v = 0; v < lp.n_versions; ++v)
          if (job_class(std::get<0>(keys[v])) == pass) vorder.push_back(v);
      if (tc_layer) {
        const LayerInfo& src = m->layers[li.d.input];
        lp.tc_kind = layer_tensor_kind(m, li);
        aiq_status_t st = lp.tc_kind == 3
            ? conv_rs_encode_maps(make_geom(m, li, B), ws + wl.slot_off[src.slot], B, plan.lp[li.d.input].n_versions, &lp.maps[0])
            : lp.tc_kind == 1
            ? conv_tc_encode_map(make_geom(m, li, B), ws + wl.slot_off[src.slot], B, plan.lp[li.d.input].n_versions, &lp.maps[0])
            : conv_pw_tc_encode_map(make_geom(m, li, B), ws + wl.slot_off[src.slot], B, plan.lp[li.d.input].n_versions, &lp.maps[0]);
        if (st != AIQ_OK) return st;
        if (lp.tc_kind == 2) {
          st = conv_pw_tc_encode_out_map(make_geom(m, li, B), ws + wl.slot_off[li.slot], B, lp.n_versions, &lp.maps[1]);
          if (st != AIQ_OK) return st;
        }
      }
      for (int v : vorder) {
        LayerJob j = {};
        const int bits = std::get<0>(keys[v]);
        const int bi = bits_index(bits);
        j.in = li.d.input >= 0 ? slot_ptr(li.d.input, std::get<1>(keys[v])) : nullptr;
        j.res = li.d.residual >= 0 ? slot_ptr(li.d.residual, std::get<2>(keys[v])) : nullptr;
        j.out = slot_ptr(l, v);
        j.in_version = li.d.input >= 0 ? std::get<1>(keys[v]) : 0;
        j.out_version = v;
        j.w = li.packed[bi];
        j.scale = li.scales[bi];
        j.bias = li.bias;
        j.bits = bits;
        if (g_opt_fuse_pool.load() && l == m->pool_layer && fuse_head[l] < 0) {
          j.pool = pooled_base + (size_t)v * B * li.d.cout;      // the row the classifier reads for this version
          lp.pools = true;
        }
        plan.jobs.push_back(j);
        const double wb = (double)li.d.cout * (row_bytes(li.K, bits) + 8.0);
        switch (job_class(bits)) {
          case 0: lp.n_tc++; lp.weight_bytes_tc += wb; break;
          case 1: lp.n_tc16++; lp.weight_bytes_tc16 += wb; break;
          case 2: lp.n_tc32++; lp.weight_bytes_tc32 += wb; break;
          default: lp.weight_bytes += wb;
        }
      }
      continue;
    }
    // classifier: pool every distinct input version once, then one linear job per version
    // (grouped by bit-width), then arg-max per version
    const LayerInfo& src = m->layers[li.d.input];
    int n_in_versions = 0;
    for (int s = 0; s < S; ++s) n_in_versions = std::max(n_in_versions, ver[li.d.input][s] + 1);
    lp.n_pool = n_in_versions;
    lp.pool_first = plan.jobs.size();
    float* pooled = reinterpret_cast<float*>(ws + wl.pooled_off);
    for (int v = 0; v < n_in_versions; ++v) {
      LayerJob j = {};
      j.in = slot_ptr(li.d.input, v);
      j.out = pooled + (size_t)v * B * src.d.cout;
      plan.jobs.push_back(j);
    }
    // order the linear jobs by bit-width so each launch is homogeneous
    std::vector<int> vorder;
    for (int b = 0; b < 4; ++b)
      for (int v = 0; v < lp.n_versions; ++v)
        if (std::get<0>(keys[v]) == kBitsList[b]) vorder.push_back(v);
    float* logits = user_logits ? user_logits : reinterpret_cast<float*>(ws + wl.logits_off);
    lp.job_first = plan.jobs.size();
    for (size_t idx = 0; idx < vorder.size(); ++idx) {
      const int v = vorder[idx];
      const int bits = std::get<0>(keys[v]);
      const int bi = bits_index(bits);
      LayerJob j = {};
      j.in = pooled + (size_t)std::get<1>(keys[v]) * B * src.d.cout;
      j.out = logits + (size_t)v * B * li.d.cout;
      j.w = li.packed[bi];
      j.scale = li.scales[bi];
      j.bias = li.bias;
      j.bits = bits;
      if (lp.group_bits.empty() || lp.group_bits.back() != bits) {
        lp.group_bits.push_back(bits);
        lp.bit_groups.push_back({(int)idx, 1});
      } else {
        lp.bit_groups.back().second++;
      }
      plan.jobs.push_back(j);
    }
    lp.argmax_first = plan.jobs.size();
    for (int v = 0; v < lp.n_versions; ++v) {
      LayerJob j = {};
      j.in = logits + (size_t)v * B * li.d.cout;
      j.label_slot = v;
      plan.jobs.push_back(j);
    }
    plan.final_version.assign(S, 0);
    for (int s = 0; s < S; ++s) plan.final_version[s] = ver[l][s];
    plan.n_final = lp.n_versions;
  }
  if (plan.jobs.size() > jobs_capacity(m, S))
    return set_error(AIQ_ERR_WORKSPACE_TOO_SMALL, "internal: job table overflow");
  return AIQ_OK;
}

// Launches one pass over a chunk of `B` images (B <= the plan's chunk size).
static aiq_status_t run_chunk(const aiq_model* m, const EvalPlan& plan, const LayerJob* jobs_dev, int B,
                              const float* x_chunk, const int32_t* labels, int32_t* counts, int32_t* preds,
                              long long preds_stride, long long img0, bool want_argmax, cudaStream_t stream) {
  for (int l : m->order) {
    const LayerInfo& li = m->layers[l];
    const LayerPlan& lp = plan.lp[l];
    aiq_status_t st;
    if (li.d.kind == AIQ_LAYER_FC) {
      const LayerInfo& src = m->layers[li.d.input];
      if (!plan.lp[li.d.input].pools) {           // else the producing layer's epilogue has written the pooled rows
        st = launch_avgpool(jobs_dev + lp.pool_first, lp.n_pool, B, src.Ho, src.Wo, src.d.cout, m->act_format, stream);
        if (st != AIQ_OK) return st;
      }
      for (size_t gi = 0; gi < lp.bit_groups.size(); ++gi) {
        const size_t first = lp.job_first + lp.bit_groups[gi].first;
        st = launch_qlinear(jobs_dev + first, &plan.jobs[first], lp.bit_groups[gi].second, li.d.cout, li.K, B, stream);
        if (st != AIQ_OK) return st;
      }
      if (want_argmax) {
        st = launch_argmax_count(jobs_dev + lp.argmax_first, lp.n_versions, B, li.d.cout, labels, counts, preds,
                                 preds_stride, img0, stream);
        if (st != AIQ_OK) return st;
      }
      continue;
    }
    if (lp.skipped) continue;
    const ConvGeom g = make_geom(m, li, B);
    if (lp.fused_head >= 0 && lp.fused_mid >= 0) {
      st = launch_mb_block(make_geom(m, m->layers[lp.fused_head], B), make_geom(m, m->layers[lp.fused_mid], B), g, li.mb_nh,
                           jobs_dev + lp.job_first, lp.n_tc, m->status_word, lp.weight_bytes_tc, stream);
      if (st != AIQ_OK) return st;
      continue;
    }
    if (lp.fused_head >= 0) {
      st = launch_conv_rs_block(g, &lp.maps[0], jobs_dev + lp.job_first, lp.n_tc, plan.batch_capacity, m->status_word,
                                lp.weight_bytes_tc, stream);
      if (st != AIQ_OK) return st;
      continue;
    }
    if (li.d.kind == AIQ_LAYER_DEPTHWISE) {
      st = launch_depthwise(g, jobs_dev + lp.job_first, lp.n_versions, x_chunk, lp.weight_bytes, stream);
      if (st != AIQ_OK) return st;
      continue;
    }
    auto launch_wide = [&](const LayerJob* jd, int n, double wb, int wbits) -> aiq_status_t {
      return lp.tc_kind == 3
          ? launch_conv_rs(g, &lp.maps[0], jd, n, plan.batch_capacity, m->status_word, wb, wbits, lp.pools, stream)
          : lp.tc_kind == 2
          ? launch_conv_pw_tc(g, &lp.maps[0], &lp.maps[1], jd, n, plan.batch_capacity, m->status_word, wb, wbits, stream)
          : launch_conv_tc(g, &lp.maps[0], jd, n, plan.batch_capacity, m->status_word, wb, wbits, stream);
    };
    if (lp.n_tc > 0) {
      st = launch_wide(jobs_dev + lp.job_first, lp.n_tc, lp.weight_bytes_tc, 8);
      if (st != AIQ_OK) return st;
    }
    int done = lp.n_tc;
    if (lp.n_tc16 > 0) {
      st = launch_wide(jobs_dev + lp.job_first + done, lp.n_tc16, lp.weight_bytes_tc16, 16);
      if (st != AIQ_OK) return st;
      done += lp.n_tc16;
    }
    if (lp.n_tc32 > 0) {
      st = launch_wide(jobs_dev + lp.job_first + done, lp.n_tc32, lp.weight_bytes_tc32, 32);
      if (st != AIQ_OK) return st;
      done += lp.n_tc32;
    }
    if (lp.n_versions > done) {
      st = launch_conv(g, jobs_dev + lp.job_first + done, lp.n_versions - done, x_chunk, lp.weight_bytes, stream);
      if (st != AIQ_OK) return st;
    }
  }
  return AIQ_OK;
}

}  // namespace aiq

namespace aiq {
// The view of the model a pass of `batch` images under `n_schemes` schemes runs on.
static const aiq_model* pick_view(const aiq_model* m, int batch, int n_schemes) {
  if (!m->small_view) return m;
  return (long long)batch * n_schemes < (long long)g_opt_small_pass.load() ? m->small_view : m;
}
}  // namespace aiq

extern "C" size_t aiq_workspace_bytes(const aiq_model_t* model, int max_batch, int max_schemes) {
  if (!model || max_batch <= 0 || max_schemes <= 0) return 0;
  size_t bytes = aiq::ws_layout(model, max_batch, max_schemes).total;
  const int small_pass = aiq::g_opt_small_pass.load();     // the small view never sees a pass of this many images
  if (model->small_view && small_pass > 0)
    bytes = std::max(bytes, aiq::ws_layout(model->small_view, std::min(max_batch, small_pass), max_schemes).total);
  return bytes;
}

extern "C" void aiq_set_small_pass_images(int image_schemes) {
  aiq::g_opt_small_pass = image_schemes > 0 ? image_schemes : 0;
}

extern "C" void aiq_set_eval_options(int chunk, int share_prefix) {
  aiq::g_opt_chunk = chunk > 0 ? chunk : 0;
  aiq::g_opt_share = share_prefix ? 1 : 0;
}

extern "C" void aiq_set_scale_granularity(int granularity) {
  aiq::g_opt_per_tensor = granularity == AIQ_SCALE_PER_TENSOR ? 1 : 0;
}

extern "C" void aiq_set_fusion(int blocks, int pool) {
  aiq::g_opt_fuse = blocks & 7;
  aiq::g_opt_fuse_pool = pool ? 1 : 0;
}

extern "C" void aiq_set_compute_path(int path) {
  aiq::g_opt_path = (path == AIQ_PATH_FP32 || path == AIQ_PATH_TENSOR || path == AIQ_PATH_TENSOR_TILES) ? path : AIQ_PATH_AUTO;
}

extern "C" void aiq_last_call_stats(int64_t* kernel_launches, int64_t* layer_evals, int64_t* layer_evals_unshared) {
  if (kernel_launches) *kernel_launches = aiq::t_launches;
  if (layer_evals) *layer_evals = aiq::t_layer_evals;
  if (layer_evals_unshared) *layer_evals_unshared = aiq::t_layer_evals_unshared;
}

static aiq_status_t forward_on_view(const aiq_model_t* model, const uint8_t* scheme_bits, const float* x,
                                    int batch, float* logits, void* workspace, size_t workspace_bytes,
                                    void* stream_);

extern "C" aiq_status_t aiq_forward(const aiq_model_t* model, const uint8_t* scheme_bits, const float* x,
                                    int batch, float* logits, void* workspace, size_t workspace_bytes,
                                    void* stream_) {
  if (!model) return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_forward: null pointer");
  return forward_on_view(batch > 0 ? aiq::pick_view(model, batch, 1) : model, scheme_bits, x, batch, logits, workspace,
                         workspace_bytes, stream_);
}

static aiq_status_t forward_on_view(const aiq_model_t* model, const uint8_t* scheme_bits, const float* x,
                                    int batch, float* logits, void* workspace, size_t workspace_bytes,
                                    void* stream_) {
  using namespace aiq;
  if (!model || !scheme_bits || !x || !logits || !workspace) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward: null pointer");
  if (batch <= 0) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward: batch=%d", batch);
  if (((uintptr_t)workspace) & 255) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward: workspace not 256-byte aligned");
  if ((((uintptr_t)x) & 15) || (((uintptr_t)logits) & 3)) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward: x must be 16-byte aligned");
  const WsLayout wl = ws_layout(model, batch, 1);
  if (workspace_bytes < wl.total)
    return set_error(AIQ_ERR_WORKSPACE_TOO_SMALL, "aiq_forward: need %zu workspace bytes, got %zu", wl.total, workspace_bytes);
  aiq_status_t st = check_device_sm100();
  if (st != AIQ_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  t_launches = 0;
  EvalPlan plan;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  st = build_plan(model, scheme_bits, 1, batch, true, ws, wl, logits, plan);
  if (st != AIQ_OK) return st;
  AIQ_CUDA_TRY(cudaMemcpyAsync(ws + wl.jobs_off, plan.jobs.data(), plan.jobs.size() * sizeof(LayerJob),
                               cudaMemcpyHostToDevice, stream));
  st = run_chunk(model, plan, reinterpret_cast<const LayerJob*>(ws + wl.jobs_off), batch, x, nullptr, nullptr,
                 nullptr, 0, 0, false, stream);
  t_layer_evals = plan.versions_total;
  t_layer_evals_unshared = (int64_t)model->layers.size();
  return st;
}

extern "C" aiq_status_t aiq_eval_schemes(const aiq_model_t* model_in, const uint8_t* schemes, int n_schemes,
                                         const float* x, const int32_t* labels, int n_images, float* acc,
                                         int32_t* correct_counts, int32_t* preds, void* workspace,
                                         size_t workspace_bytes, void* stream_) {
  using namespace aiq;
  const aiq_model_t* model = model_in;
  if (model_in && n_schemes > 0 && n_images > 0) {
    const int want = g_opt_chunk.load() > 0 ? g_opt_chunk.load() : 1024;
    model = pick_view(model_in, std::min(want, n_images), n_schemes);
  }
  if (!model || !schemes || !x || !labels || !acc || !workspace)
    return set_error(AIQ_ERR_INVALID_ARG, "aiq_eval_schemes: null pointer");
  if (n_schemes <= 0 || n_images <= 0)
    return set_error(AIQ_ERR_INVALID_ARG, "aiq_eval_schemes: n_schemes=%d n_images=%d", n_schemes, n_images);
  if (((uintptr_t)workspace) & 255) return set_error(AIQ_ERR_INVALID_ARG, "aiq_eval_schemes: workspace not 256-byte aligned");
  if (((uintptr_t)x) & 15) return set_error(AIQ_ERR_INVALID_ARG, "aiq_eval_schemes: x must be 16-byte aligned");
  aiq_status_t st = check_device_sm100();
  if (st != AIQ_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  t_launches = 0;

  // chunk: the requested (or default) size, shrunk until the layout fits the workspace
  const int opt_chunk = g_opt_chunk.load();
  int B = opt_chunk > 0 ? opt_chunk : 1024;
  if (B > n_images) B = n_images;
  while (B > 1 && ws_layout(model, B, n_schemes).total > workspace_bytes) B = (B + 1) / 2;
  const WsLayout wl = ws_layout(model, B, n_schemes);
  if (wl.total > workspace_bytes)
    return set_error(AIQ_ERR_WORKSPACE_TOO_SMALL, "aiq_eval_schemes: need %zu workspace bytes for one image, got %zu",
                     wl.total, workspace_bytes);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  EvalPlan plan;
  st = build_plan(model, schemes, n_schemes, B, g_opt_share.load() != 0, ws, wl, nullptr, plan);
  if (st != AIQ_OK) return st;
  // Counts and predictions are indexed by a row in [0, n_schemes): the row of a final
  // version is the first scheme that maps to it; duplicate schemes are filled in afterwards.
  std::vector<int> first_scheme(plan.n_final, -1);
  for (int s = 0; s < n_schemes; ++s)
    if (first_scheme[plan.final_version[s]] < 0) first_scheme[plan.final_version[s]] = s;
  const LayerPlan& fcp = plan.lp.back();
  for (int v = 0; v < plan.n_final; ++v) plan.jobs[fcp.argmax_first + v].label_slot = first_scheme[v];

  int32_t* counts_dev = reinterpret_cast<int32_t*>(ws + wl.counts_off);
  AIQ_CUDA_TRY(cudaMemcpyAsync(ws + wl.jobs_off, plan.jobs.data(), plan.jobs.size() * sizeof(LayerJob),
                               cudaMemcpyHostToDevice, stream));
  AIQ_CUDA_TRY(cudaMemsetAsync(counts_dev, 0, (size_t)n_schemes * 4, stream));

  const size_t img_elems = (size_t)model->in_c * model->in_h * model->in_w;
  const LayerJob* jobs_dev = reinterpret_cast<const LayerJob*>(ws + wl.jobs_off);
  int64_t chunks = 0;
  for (long long img0 = 0; img0 < n_images; img0 += B, ++chunks) {
    const int b = (int)std::min<long long>(B, n_images - img0);
    st = run_chunk(model, plan, jobs_dev, b, x + img0 * img_elems, labels, counts_dev, preds, n_images, img0, true, stream);
    if (st != AIQ_OK) return st;
  }
  std::vector<int32_t> counts(n_schemes, 0);
  AIQ_CUDA_TRY(cudaMemcpyAsync(counts.data(), counts_dev, (size_t)n_schemes * 4, cudaMemcpyDeviceToHost, stream));
  if (preds)
    for (int s = 0; s < n_schemes; ++s) {
      const int src = first_scheme[plan.final_version[s]];
      if (src != s)
        AIQ_CUDA_TRY(cudaMemcpyAsync(preds + (size_t)s * n_images, preds + (size_t)src * n_images,
                                     (size_t)n_images * 4, cudaMemcpyDeviceToDevice, stream));
    }
  int32_t dev_status = 0;
  AIQ_CUDA_TRY(cudaMemcpyAsync(&dev_status, model->status_word, 4, cudaMemcpyDeviceToHost, stream));
  AIQ_CUDA_TRY(cudaStreamSynchronize(stream));
  if (dev_status) {
    AIQ_CUDA_TRY(cudaMemsetAsync(model->status_word, 0, 4, stream));
    return set_error(AIQ_ERR_TIMEOUT, "aiq_eval_schemes: a bounded wait inside a kernel expired; results are invalid");
  }
  for (int s = 0; s < n_schemes; ++s) {
    const int c = counts[first_scheme[plan.final_version[s]]];
    acc[s] = (float)((double)c / (double)n_images);
    if (correct_counts) correct_counts[s] = c;
  }
  t_layer_evals = plan.versions_total * chunks;
  t_layer_evals_unshared = (int64_t)n_schemes * (int64_t)model->layers.size() * chunks;
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// aiq_forward for callers that have no device memory to lend as workspace.
//
// The workspace of this variant is a fixed array that is part of the library image: every
// GPU that loads the library keeps AIQ_STATIC_WORKSPACE_BYTES of it until the process ends.
// In host code the array's name is only a handle for the runtime, not a device address, so
// the address is looked up once per device with cudaGetSymbolAddress and that pointer is
// what the kernels receive.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[AIQ_STATIC_WORKSPACE_BYTES];

namespace aiq {
// Device address of the array per device; nullptr until the first call on that device.  Two
// host threads that make their first call at the same time both look the address up and
// publish the same value, which is harmless; the atomic only makes sure that a reader never
// sees a half-published pointer.
static std::atomic<void*> g_static_ws_ptr[64];
}  // namespace aiq

extern "C" aiq_status_t aiq_forward_static(const aiq_model_t* model, const uint8_t* scheme_bits,
                                           const float* x, int batch, float* logits, void* stream_) {
  using namespace aiq;
  if (!model || !scheme_bits || !x || !logits)
    return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward_static: null pointer");
  if (batch <= 0) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward_static: batch=%d", batch);
  const size_t need = ws_layout(model, batch, 1).total;
  if (need > (size_t)AIQ_STATIC_WORKSPACE_BYTES)
    return set_error(AIQ_ERR_WORKSPACE_TOO_SMALL,
                     "aiq_forward_static: batch %d of this model needs %zu workspace bytes, the built-in "
                     "workspace holds %zu; use a smaller batch or aiq_forward with your own workspace",
                     batch, need, (size_t)AIQ_STATIC_WORKSPACE_BYTES);
  aiq_status_t st = check_device_sm100();
  if (st != AIQ_OK) return st;
  int dev = 0;
  AIQ_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return set_error(AIQ_ERR_INVALID_ARG, "aiq_forward_static: device %d", dev);
  void* ws_ptr = g_static_ws_ptr[dev].load(std::memory_order_acquire);
  if (!ws_ptr) {
    // first call on this device (it is the current one): resolve the array's device address
    cudaError_t e = cudaGetSymbolAddress(&ws_ptr, g_static_workspace);
    if (e != cudaSuccess || !ws_ptr)
      return set_error(AIQ_ERR_CUDA, "cudaGetSymbolAddress(static workspace): %s", cudaGetErrorString(e));
    g_static_ws_ptr[dev].store(ws_ptr, std::memory_order_release);
  }
  // Nothing in the workspace has to start at zero for a forward pass: the job records are
  // copied in, and every activation, pooled value and logit is written before it is read.
  return forward_on_view(model, scheme_bits, x, batch, logits, ws_ptr,
                     (size_t)AIQ_STATIC_WORKSPACE_BYTES, stream_);
}

// ---------------------------------------------------------------------------------------
// analytic arithmetic intensity (host only)
// ---------------------------------------------------------------------------------------
extern "C" aiq_status_t aiq_scheme_ai(const aiq_model_t* model, const uint8_t* scheme_bits, int ai_batch,
                                      double* ai, double* flops, double* bytes) {
  using namespace aiq;
  if (!model || !scheme_bits) return set_error(AIQ_ERR_INVALID_ARG, "aiq_scheme_ai: null pointer");
  if (ai_batch <= 0) return set_error(AIQ_ERR_INVALID_ARG, "aiq_scheme_ai: ai_batch=%d", ai_batch);
  double fl = 0.0, by = 0.0;
  for (size_t l = 0; l < model->layers.size(); ++l) {
    const LayerInfo& li = model->layers[l];
    const int bits = scheme_bits[l];
    if (!bits_ok(bits)) return set_error(AIQ_ERR_UNSUPPORTED_BITS, "aiq_scheme_ai: layer %zu bits=%d", l, bits);
    const double weights = (double)li.d.cout * li.K;
    fl += 2.0 * weights * li.Ho * li.Wo * ai_batch;
    by += weights * bits / 8.0;
    by += 4.0 * ai_batch * ((double)li.d.cin * li.Hi * li.Wi + (double)li.d.cout * li.Ho * li.Wo);
  }
  if (ai) *ai = fl / by;
  if (flops) *flops = fl;
  if (bytes) *bytes = by;
  return AIQ_OK;
}

extern "C" aiq_status_t aiq_profile_start(void) {
  using namespace aiq;
  if (!t_prof) t_prof = new std::vector<ProfiledLaunch>();
  if (!t_event_pool) t_event_pool = new std::vector<cudaEvent_t>();
  for (ProfiledLaunch& pl : *t_prof) { t_event_pool->push_back(pl.start); t_event_pool->push_back(pl.stop); }
  t_prof->clear();
  memset(t_work, 0, sizeof(t_work));
  t_profiling = true;
  return AIQ_OK;
}

extern "C" aiq_status_t aiq_profile_stop(aiq_kernel_profile_t* out) {
  using namespace aiq;
  if (!out) return set_error(AIQ_ERR_INVALID_ARG, "aiq_profile_stop: null pointer");
  if (!t_profiling) return set_error(AIQ_ERR_INVALID_ARG, "aiq_profile_stop without aiq_profile_start");
  t_profiling = false;
  for (int k = 0; k < AIQ_KERNEL_KINDS; ++k) { out[k] = t_work[k]; out[k].ms = 0.0; }
  for (ProfiledLaunch& pl : *t_prof) {
    AIQ_CUDA_TRY(cudaEventSynchronize(pl.stop));
    float ms = 0.f;
    AIQ_CUDA_TRY(cudaEventElapsedTime(&ms, pl.start, pl.stop));
    out[pl.kind].ms += ms;
  }
  for (ProfiledLaunch& pl : *t_prof) { t_event_pool->push_back(pl.start); t_event_pool->push_back(pl.stop); }
  t_prof->clear();
  return AIQ_OK;
}

extern "C" const char* aiq_status_string(aiq_status_t status) {
  switch (status) {
    case AIQ_OK: return "ok";
    case AIQ_ERR_INVALID_ARG: return "invalid argument";
    case AIQ_ERR_UNSUPPORTED_BITS: return "unsupported bit-width";
    case AIQ_ERR_SHAPE: return "shape mismatch";
    case AIQ_ERR_WORKSPACE_TOO_SMALL: return "buffer too small";
    case AIQ_ERR_CUDA: return "CUDA error";
    case AIQ_ERR_NOT_SM100: return "device is not sm_100";
    case AIQ_ERR_NONFINITE: return "non-finite weight";
    case AIQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" const char* aiq_last_error(void) { return aiq::t_err; }
