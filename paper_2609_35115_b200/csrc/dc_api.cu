// C ABI of the streaming decoder step: model / stream lifetime, admission checks and the host
// side of one chunk step.  Every step of the path runs in the kernels; this file only validates,
// sizes the address-stable state and enqueues launches.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <new>
#include <string>
#include <map>
#include <vector>

#include "dc_internal.h"

namespace dc {

static thread_local std::string g_last_error;

void set_error(const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  g_last_error = buf;
}

// ---- device allocation shim (see dc_internal.h) ---------------------------------------------------------------
namespace {
constexpr size_t   kGuardBytes = 256;
constexpr int      kGuardByte = 0xC5;
struct GuardInfo { void* base; size_t bytes; };
std::mutex g_guard_mu;
std::map<void*, GuardInfo> g_guarded;          // user pointer -> allocation with guard zones
thread_local int  g_fail_countdown = 0;         // > 0: the allocation that brings it to 0 fails
thread_local bool g_guard_mode = false;
}  // namespace

cudaError_t dev_alloc(void** p, size_t bytes) {
  *p = nullptr;
  if (g_fail_countdown > 0 && --g_fail_countdown == 0) return cudaErrorMemoryAllocation;   // injected: the device is not touched
  if (!g_guard_mode) return cudaMalloc(p, bytes);
  void* base = nullptr;
  cudaError_t e = cudaMalloc(&base, bytes + 2 * kGuardBytes);
  if (e != cudaSuccess) return e;
  char* user = static_cast<char*>(base) + kGuardBytes;
  e = cudaMemset(base, kGuardByte, kGuardBytes);
  if (e == cudaSuccess) e = cudaMemset(user + bytes, kGuardByte, kGuardBytes);
  if (e != cudaSuccess) {
    cudaFree(base);
    return e;
  }
  {
    std::lock_guard<std::mutex> lk(g_guard_mu);
    g_guarded[user] = GuardInfo{base, bytes};
  }
  *p = user;
  return cudaSuccess;
}

void dev_free(void* p) {
  if (!p) return;
  {
    std::lock_guard<std::mutex> lk(g_guard_mu);
    auto it = g_guarded.find(p);
    if (it != g_guarded.end()) {
      p = it->second.base;
      g_guarded.erase(it);
    }
  }
  cudaFree(p);
}

// Reads the guard zones of one allocation back; returns the number of zones (0..2) whose pattern changed, or -1 on a
// CUDA error.  An allocation without guard zones counts as intact.
static int damaged_guards(const void* user) {
  GuardInfo gi{};
  {
    std::lock_guard<std::mutex> lk(g_guard_mu);
    auto it = g_guarded.find(const_cast<void*>(user));
    if (it == g_guarded.end()) return 0;
    gi = it->second;
  }
  unsigned char h[2 * kGuardBytes];
  if (cudaMemcpy(h, gi.base, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(h + kGuardBytes, static_cast<const char*>(user) + gi.bytes, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
    return -1;
  int bad = 0;
  for (int z = 0; z < 2; ++z)
    for (size_t i = 0; i < kGuardBytes; ++i)
      if (h[z * kGuardBytes + i] != kGuardByte) {
        ++bad;
        break;
      }
  return bad;
}

#define DC_CUDA(expr)                                                                    \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess) {                                                            \
      dc::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
      return e__ == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;                \
    }                                                                                    \
  } while (0)

static int pow2_ceil(int v) {
  int p = 1;
  while (p < v) p <<= 1;
  return p;
}

// One fp32 layer of the conv pipeline / vocoder tail.
struct F32Layer {
  int    kind;        // 0 conv k3, 1 transposed conv, 2 head + iSTFT
  int    C_in, C_out;
  int    dil;         // conv dilation
  int    stride;      // transposed conv stride
  int    rate_in;     // input frames of this layer per chunk frame
  int    halo;        // left-context frames it reads
  int    residual_silu, post_silu;
  size_t w_off, b_off;  // float offsets in the blob
  int    ring_cap;    // rows of its input ring
  int    excite;      // the random excitation is added to this layer's output
};

}  // namespace dc

using dc::DevBuf;
using dc::F32Layer;

struct dc_model {
  dc_config cfg;
  int       device = 0;
  float*    d_w = nullptr;   // fp32 pipelines: the blob on the device
  // flow pipeline: staging of dc_decode_batch_host (pinned host + device, max_batch chunks each way)
  float *h_in = nullptr, *h_out = nullptr, *d_in = nullptr, *d_out = nullptr;
  bool   zero_copy = true;   // dc_decode_batch_host: kernels access page-locked caller buffers directly
  int*   h_err = nullptr;   // pinned: the device error word, read back by the host-buffer calls
  std::vector<F32Layer> layers;
  int       out_per_frame = 0;
  int       in_dim = 0;
  dc::FlowModel* flow = nullptr;
  // DC_PIPE_TOKEN2WAV: the flow decoder and the vocoder tail as models of their own; this one only chains them
  dc_model* sub_flow = nullptr;
  dc_model* sub_voc = nullptr;
  // fp32 pipelines: dc_decode_batch runs every layer ONCE for all the streams of the batch (slot = grid plane); the slot
  // records live here and are rewritten per call by the first node of the captured batch step
  dc::F32Batch*   d_batch = nullptr;
  cudaGraph_t     gb_graph = nullptr;
  cudaGraphExec_t gb_exec = nullptr;
  cudaGraphNode_t gb_set_node = nullptr;
  int             gb_launches = 0;
  std::atomic<uint64_t> counters[8];
  std::atomic<int> open_streams{0};
  int    streams_opened = 0;   // so far: the next fp32 stream's random-stream index (streams of a model are opened one at a time)
  std::mutex mu;
  dc::Profiler prof;
  std::vector<dc_stream*> all_streams;   // host structs live until dc_destroy, so a closed handle stays detectable
};

static void free_batch_graph(dc_model* m) {
  if (m->gb_exec) cudaGraphExecDestroy(m->gb_exec);
  if (m->gb_graph) cudaGraphDestroy(m->gb_graph);
  if (m->d_batch) dc::dev_free(m->d_batch);
  m->gb_exec = nullptr;
  m->gb_graph = nullptr;
  m->d_batch = nullptr;
}

struct dc_stream {
  dc_model* model = nullptr;
  bool      closed = false, poisoned = false;
  long long frames_total = 0;
  long long chunks = 0;
  int       rng_id = 0;            // fp32 pipelines: which device random stream the session draws from (vocoder excitation)
  std::vector<DevBuf> f32_rings;   // input ring of each fp32 layer
  float*    tails = nullptr;       // [2][12] overlap-add tails (ping-pong)
  dc::F32StreamPtrs* d_ptrs = nullptr;   // fp32 pipelines: the addresses of this stream's rings and tails, for batched launches
  dc::F32Call* d_call = nullptr;   // fp32 pipelines: per-call record read by this stream's captured graph (streams of one
                                   // model may decode at the same time on different CUDA streams)
  dc::FlowState* flow = nullptr;
  dc_stream* sub_flow = nullptr;   // DC_PIPE_TOKEN2WAV: the two halves' streams and the mel chunk between them
  dc_stream* sub_voc = nullptr;
  float*    mel = nullptr;         // [f_chunk][mel_dim] fp32, device
  float*    wave_mel = nullptr;    // dc_decode_wavefront of the composite: all mel frames of one call (max_wave_frames rows, sized at open)
  long long wave_mel_frames = 0;
  cudaStream_t wave_side = nullptr;   // the vocoder tail of a wavefront call runs here, beside the flow decoder's passes
  cudaEvent_t  wave_ev = nullptr;
  float*    stage_in = nullptr;    // device staging of dc_decode_chunk_host
  float*    stage_out = nullptr;
  cudaGraph_t     g_graph = nullptr;   // fp32 pipelines: the captured chunk step
  cudaGraphExec_t g_exec = nullptr;
  cudaGraphNode_t g_set_node = nullptr;
  int             g_launches = 0;
};

// ---------------------------------------------------------------------------------------------
// configuration
// ---------------------------------------------------------------------------------------------

static dc_config sub_config(const dc_config& c, int pipeline) {
  dc_config s = c;
  s.pipeline = pipeline;
  s.precision = pipeline == DC_PIPE_FLOW ? DC_BF16 : DC_F32;
  s.max_wave_frames = 0;   // the mel buffer of a wavefront call belongs to the composite
  if (pipeline == DC_PIPE_FLOW) {
    s.excitation_std = 0.f;
    s.excitation_seed_lo = s.excitation_seed_hi = 0;
  }
  if (pipeline != DC_PIPE_FLOW) {
    s.cfg_scale = 0.f;
    s.f_prompt = 0;
    s.f_lookahead = 0;
    s.noise_seed_lo = s.noise_seed_hi = 0;
  }
  return s;
}

static bool config_ok(const dc_config* c, const char** why) {
#define BAD(msg) do { *why = msg; return false; } while (0)
  if (!c) BAD("null config");
  if (c->size != sizeof(dc_config)) BAD("dc_config.size mismatch");
  if (c->f_chunk < 1 || c->f_chunk > 4096) BAD("f_chunk out of range");
  if (c->max_batch < 1 || c->max_batch > 1024) BAD("max_batch out of range");
  if (!(c->cfg_scale >= 0.f && c->cfg_scale <= 100.f)) BAD("cfg_scale out of range");
  if (c->f_prompt < 0 || c->f_prompt > 4096) BAD("f_prompt out of range");
  if (c->f_lookahead < 0 || c->f_lookahead > 32) BAD("f_lookahead out of range");
  if ((c->noise_seed_lo | c->noise_seed_hi) != 0 && c->pipeline != DC_PIPE_FLOW && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("noise_seed belongs to the flow decoder");
  if (c->f_lookahead != 0 && c->pipeline != DC_PIPE_FLOW && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("f_lookahead belongs to the flow decoder");
  if (c->f_prompt != 0 && c->pipeline != DC_PIPE_FLOW && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("f_prompt belongs to the flow decoder");
  if (c->cfg_scale != 0.f && c->pipeline != DC_PIPE_FLOW && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("cfg_scale belongs to the flow decoder");
  if (c->options & ~(uint32_t)(DC_OPT_NO_GRAPH | DC_OPT_NO_PDL | DC_OPT_NO_ZEROCOPY | DC_OPT_SERIAL_TAILS | DC_OPT_ROUNDED_NORM | DC_OPT_SKIP_CONV_GEMM |
                               DC_OPT_SKIP_ATTENTION | DC_OPT_EMPTY_KERNELS | DC_OPT_GUARD_ZONES | DC_OPT_CTA_PAIRS))
    BAD("unknown option bit");
  if (!(c->excitation_std >= 0.f && c->excitation_std <= 1e6f)) BAD("excitation_std out of range");
  if (c->excitation_std > 0.f && c->pipeline != DC_PIPE_VOCODER && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("excitation_std belongs to the vocoder tail");
  if (c->excitation_std > 0.f && (c->excitation_seed_lo | c->excitation_seed_hi) == 0) BAD("excitation_std > 0 needs a non-zero excitation seed");
  if (c->max_wave_frames < 0 || c->max_wave_frames > (1 << 24)) BAD("max_wave_frames out of range");
  if (c->max_wave_frames != 0 && c->pipeline != DC_PIPE_TOKEN2WAV) BAD("max_wave_frames belongs to the token2wav pipeline");
  if (c->pipeline == DC_PIPE_TOKEN2WAV) {
    if (c->precision != DC_BF16) BAD("token2wav pipeline is bf16 (flow decoder) + fp32 (vocoder tail)");
    const dc_config f = sub_config(*c, DC_PIPE_FLOW), v = sub_config(*c, DC_PIPE_VOCODER);
    return config_ok(&f, why) && config_ok(&v, why);
  }
  if ((c->pipeline == DC_PIPE_CONV || c->pipeline == DC_PIPE_VOCODER) && c->max_batch > dc::F32_MAX_BATCH) BAD("fp32 pipelines batch at most 64 streams");
  if (c->pipeline == DC_PIPE_CONV) {
    if (c->precision != DC_F32) BAD("conv pipeline is fp32");
    if (c->hidden < 4 || c->hidden % 4) BAD("hidden must be a multiple of 4");
    if (c->n_conv < 1 || c->n_conv > DC_MAX_CONV) BAD("n_conv out of range");
    for (int l = 0; l < c->n_conv; ++l)
      if (c->dilations[l] < 1 || c->dilations[l] > 64) BAD("dilation out of range");
  } else if (c->pipeline == DC_PIPE_FLOW) {
    if (c->precision != DC_BF16) BAD("flow pipeline is bf16");
    if (c->hidden < 64 || c->hidden % 64 || c->hidden > 2048) BAD("hidden must be a multiple of 64");
    if (c->n_conv < 1 || c->n_conv > DC_MAX_CONV) BAD("n_conv out of range");
    for (int l = 0; l < c->n_conv; ++l)
      if (c->dilations[l] < 1 || c->dilations[l] > 4) BAD("flow conv dilation must be 1..4");
    if (c->n_attn < 0 || (c->n_attn > 0 && c->n_conv % c->n_attn)) BAD("n_conv must be a multiple of n_attn");
    if (c->n_attn > 0) {
      if (c->head_dim != 32 && c->head_dim != 64) BAD("head_dim must be 32 or 64");
      if (c->n_heads * c->head_dim != c->hidden) BAD("n_heads * head_dim != hidden");
      if (c->kv_cap < 1 || c->kv_cap > 4096) BAD("kv_cap out of range");
    }
    if (c->n_steps < 1 || c->n_steps > 64) BAD("n_steps out of range");
    if (c->mel_dim < 16 || c->mel_dim % 16 || c->mel_dim > 128) BAD("mel_dim must be a multiple of 16, <= 128");
    if (c->f_chunk + c->f_lookahead > 56) BAD("flow f_chunk + f_lookahead must be <= 56");
  } else if (c->pipeline == DC_PIPE_VOCODER) {
    if (c->precision != DC_F32) BAD("vocoder pipeline is fp32");
    if (c->mel_dim < 4 || c->mel_dim % 4) BAD("mel_dim must be a multiple of 4");
    if (c->n_up < 1 || c->n_up > DC_MAX_UP) BAD("n_up out of range");
    int up = 1;
    for (int q = 0; q < c->n_up; ++q) {
      if (c->up_strides[q] < 1 || c->up_strides[q] > 16) BAD("stride out of range");
      up *= c->up_strides[q];
    }
    if (up < 3) BAD("total upsampling must be >= 3");
    for (int q = 0; q <= c->n_up; ++q)
      if (c->up_channels[q] < 4 || c->up_channels[q] % 4) BAD("channels must be multiples of 4");
    if (c->n_res < 0 || c->n_res > DC_MAX_RES) BAD("n_res out of range");
    for (int r = 0; r < c->n_res; ++r)
      if (c->res_dilations[r] < 1 || c->res_dilations[r] > 64) BAD("dilation out of range");
    if (c->n_fft != 16 || c->hop != 4) BAD("only n_fft = 16, hop = 4 is built");
    if ((long long)c->f_chunk * up > (1 << 20)) BAD("chunk too long");
  } else {
    BAD("unknown pipeline");
  }
#undef BAD
  return true;
}

extern "C" size_t dc_weights_count(const dc_config* c) {
  const char* why = "";
  if (!config_ok(c, &why)) return 0;
  size_t n = 0;
  const size_t C = (size_t)c->hidden;
  if (c->pipeline == DC_PIPE_TOKEN2WAV) {
    const dc_config f = sub_config(*c, DC_PIPE_FLOW), v = sub_config(*c, DC_PIPE_VOCODER);
    return dc_weights_count(&f) + dc_weights_count(&v);
  }
  if (c->pipeline == DC_PIPE_CONV) {
    n = (size_t)c->n_conv * (3 * C * C + C);
  } else if (c->pipeline == DC_PIPE_FLOW) {
    const size_t m = (size_t)c->mel_dim;
    n = 2 * m * C + C + (size_t)c->n_conv * (3 * C * C + C + C * C) + (size_t)c->n_attn * (4 * C * C + 4 * C) + C * m + m;
  } else {
    n = 3 * (size_t)c->mel_dim * c->up_channels[0] + c->up_channels[0];
    for (int q = 0; q < c->n_up; ++q) {
      const size_t ci = c->up_channels[q], co = c->up_channels[q + 1];
      n += 2 * (size_t)c->up_strides[q] * ci * co + co + (size_t)c->n_res * (3 * co * co + co);
    }
    n += 3 * (size_t)c->up_channels[c->n_up] * (c->n_fft + 2) + (c->n_fft + 2);
  }
  return n;
}

static void build_f32_layers(dc_model* m) {
  const dc_config& c = m->cfg;
  size_t off = 0;
  auto add = [&](int kind, int ci, int co, int dil, int stride, int rate_in, int halo, int res, size_t wsz) {
    F32Layer L{};
    L.kind = kind; L.C_in = ci; L.C_out = co; L.dil = dil; L.stride = stride;
    L.rate_in = rate_in; L.halo = halo; L.residual_silu = res; L.post_silu = 0;
    L.w_off = off; off += wsz;
    L.b_off = off; off += (size_t)co;
    L.ring_cap = dc::pow2_ceil(c.f_chunk * rate_in + halo);
    m->layers.push_back(L);
  };
  if (c.pipeline == DC_PIPE_CONV) {
    const int C = c.hidden;
    for (int l = 0; l < c.n_conv; ++l) add(0, C, C, c.dilations[l], 1, 1, 2 * c.dilations[l], 1, (size_t)3 * C * C);
    m->in_dim = C;
    m->out_per_frame = C;
  } else {
    int rate = 1;
    add(0, c.mel_dim, c.up_channels[0], 1, 1, rate, 2, 0, (size_t)3 * c.mel_dim * c.up_channels[0]);
    for (int q = 0; q < c.n_up; ++q) {
      const int ci = c.up_channels[q], co = c.up_channels[q + 1], s = c.up_strides[q];
      add(1, ci, co, 1, s, rate, 1, 0, (size_t)2 * s * ci * co);
      if (q == c.n_up - 1 && c.excitation_std > 0.f) m->layers.back().excite = 1;
      rate *= s;
      for (int r = 0; r < c.n_res; ++r)
        add(0, co, co, c.res_dilations[r], 1, rate, 2 * c.res_dilations[r], 1, (size_t)3 * co * co);
    }
    m->layers.back().post_silu = 1;   // only the head reads it, and the head wants SiLU(a)
    add(2, c.up_channels[c.n_up], c.n_fft + 2, 1, 1, rate, 2, 0, (size_t)3 * c.up_channels[c.n_up] * (c.n_fft + 2));
    m->in_dim = c.mel_dim;
    m->out_per_frame = rate * c.hop;
  }
}

static void build_f32_graph(dc_stream* s);
static void build_f32_batch_graph(dc_model* m);

// ---------------------------------------------------------------------------------------------
// lifetime
// ---------------------------------------------------------------------------------------------

extern "C" dc_status dc_create(const float* w, size_t n_floats, const dc_config* cfg, dc_model** out) {
  if (!out) return DC_ERR_ARG;
  *out = nullptr;
  const char* why = "";
  if (!config_ok(cfg, &why)) {
    dc::set_error("invalid configuration: %s", why);
    return DC_ERR_CONFIG;
  }
  if (!w || n_floats != dc_weights_count(cfg)) {
    dc::set_error("weight blob has %zu floats, configuration needs %zu", n_floats, dc_weights_count(cfg));
    return DC_ERR_ARG;
  }
  int dev = 0;
  DC_CUDA(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  DC_CUDA(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) {
    dc::set_error("device %d is sm_%d%d; this library is built for sm_100a only", dev, prop.major, prop.minor);
    return DC_ERR_CUDA;
  }
  dc_model* m = new (std::nothrow) dc_model();
  if (!m) return DC_ERR_OOM;
  m->cfg = *cfg;
  m->device = dev;
  for (auto& c : m->counters) c = 0;
  dc_status st = DC_OK;
  if (cfg->pipeline == DC_PIPE_TOKEN2WAV) {
    dc_config f = sub_config(*cfg, DC_PIPE_FLOW);
    const dc_config v = sub_config(*cfg, DC_PIPE_VOCODER);
    f.options |= DC_OPT_ROUNDED_NORM;   // the vocoder tail expands the flow stage's deviation: keep every declared rounding
    const size_t nf = dc_weights_count(&f);
    st = dc_create(w, nf, &f, &m->sub_flow);
    if (st == DC_OK) st = dc_create(w + nf, n_floats - nf, &v, &m->sub_voc);
    if (st == DC_OK) {
      m->in_dim = m->sub_flow->in_dim;
      m->out_per_frame = m->sub_voc->out_per_frame;
    }
  } else if (cfg->pipeline == DC_PIPE_FLOW) {
    st = dc::flow_model_create(*cfg, w, &m->flow);
    m->in_dim = (cfg->noise_seed_lo | cfg->noise_seed_hi) ? cfg->mel_dim : 2 * cfg->mel_dim;   // [mu | x_0], or mu alone
    m->out_per_frame = cfg->mel_dim;
    if (st == DC_OK) {
      const size_t ni = (size_t)cfg->max_batch * (cfg->f_chunk + cfg->f_lookahead) * m->in_dim,
                   no = (size_t)cfg->max_batch * cfg->f_chunk * m->out_per_frame;
      cudaError_t e = cudaMallocHost(&m->h_in, ni * sizeof(float));
      if (e == cudaSuccess) e = cudaMallocHost(&m->h_out, no * sizeof(float));
      if (e == cudaSuccess) e = cudaMallocHost(&m->h_err, sizeof(int));
      m->zero_copy = !(cfg->options & DC_OPT_NO_ZEROCOPY);
      if (e == cudaSuccess) e = dc::dev_alloc(&m->d_in, ni * sizeof(float));
      if (e == cudaSuccess) e = dc::dev_alloc(&m->d_out, no * sizeof(float));
      if (e != cudaSuccess) {
        dc::set_error("staging allocation failed: %s", cudaGetErrorString(e));
        st = DC_ERR_OOM;
      }
    }
  } else {
    build_f32_layers(m);
    cudaError_t e = dc::dev_alloc(&m->d_w, n_floats * sizeof(float));
    if (e == cudaSuccess) e = cudaMemcpy(m->d_w, w, n_floats * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = dc::prepare_f32_constants();
    if (e == cudaSuccess && cfg->max_batch > 1) {
      e = dc::dev_alloc(&m->d_batch, sizeof(dc::F32Batch));
      if (e == cudaSuccess) e = cudaMemset(m->d_batch, 0, sizeof(dc::F32Batch));
    }
    if (e != cudaSuccess) {
      dc::set_error("weight upload failed: %s", cudaGetErrorString(e));
      st = e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
    }
    if (st == DC_OK && m->d_batch) build_f32_batch_graph(m);
  }
  if (st == DC_OK && !m->flow && m->h_in == nullptr) {
    // bounce buffers of dc_decode_batch_host for the pipelines whose kernels do not read host memory themselves
    // (pinned host + device, max_batch chunks each way), sized once here
    const size_t ni = (size_t)cfg->max_batch * (cfg->f_chunk + cfg->f_lookahead) * m->in_dim,
                 no = (size_t)cfg->max_batch * cfg->f_chunk * m->out_per_frame;
    cudaError_t e = cudaMallocHost(&m->h_in, ni * sizeof(float));
    if (e == cudaSuccess) e = cudaMallocHost(&m->h_out, no * sizeof(float));
    if (e == cudaSuccess) e = dc::dev_alloc(&m->d_in, ni * sizeof(float));
    if (e == cudaSuccess) e = dc::dev_alloc(&m->d_out, no * sizeof(float));
    if (e != cudaSuccess) {
      cudaGetLastError();
      dc::set_error("staging allocation failed: %s", cudaGetErrorString(e));
      st = DC_ERR_OOM;
    }
  }
  if (st != DC_OK) {
    if (m->sub_flow) dc_destroy(m->sub_flow);
    if (m->sub_voc) dc_destroy(m->sub_voc);
    free_batch_graph(m);
    if (m->d_w) dc::dev_free(m->d_w);
    if (m->flow) dc::flow_model_destroy(m->flow);
    if (m->h_in) cudaFreeHost(m->h_in);
    if (m->h_out) cudaFreeHost(m->h_out);
    if (m->h_err) cudaFreeHost(m->h_err);
    if (m->d_in) dc::dev_free(m->d_in);
    if (m->d_out) dc::dev_free(m->d_out);
    delete m;
    return st;
  }
  *out = m;
  return DC_OK;
}

extern "C" dc_status dc_destroy(dc_model* m) {
  if (!m) return DC_ERR_ARG;
  if (m->open_streams.load() != 0) {
    dc::set_error("dc_destroy: %d streams still open", m->open_streams.load());
    return DC_ERR_STATE;
  }
  if (m->sub_flow) dc_destroy(m->sub_flow);   // their streams were closed with ours
  if (m->sub_voc) dc_destroy(m->sub_voc);
  free_batch_graph(m);
  if (m->flow) dc::flow_model_destroy(m->flow);
  if (m->d_w) dc::dev_free(m->d_w);
  if (m->h_in) cudaFreeHost(m->h_in);
  if (m->h_out) cudaFreeHost(m->h_out);
  if (m->h_err) cudaFreeHost(m->h_err);
  if (m->d_in) dc::dev_free(m->d_in);
  if (m->d_out) dc::dev_free(m->d_out);
  for (dc_stream* s : m->all_streams) delete s;
  delete m;
  return DC_OK;
}

static void free_stream_buffers(dc_stream* s) {
  if (s->g_exec) cudaGraphExecDestroy(s->g_exec);
  if (s->g_graph) cudaGraphDestroy(s->g_graph);
  s->g_exec = nullptr;
  s->g_graph = nullptr;
  for (auto& b : s->f32_rings)
    if (b.p) dc::dev_free(b.p);
  s->f32_rings.clear();
  if (s->tails) dc::dev_free(s->tails);
  if (s->d_call) dc::dev_free(s->d_call);
  s->d_call = nullptr;
  if (s->d_ptrs) dc::dev_free(s->d_ptrs);
  s->d_ptrs = nullptr;
  if (s->flow) dc::flow_state_close(s->flow);
  if (s->sub_flow) dc_stream_close(s->sub_flow);
  if (s->sub_voc) dc_stream_close(s->sub_voc);
  if (s->mel) dc::dev_free(s->mel);
  if (s->wave_mel) dc::dev_free(s->wave_mel);
  s->wave_mel = nullptr;
  if (s->wave_side) cudaStreamDestroy(s->wave_side);
  if (s->wave_ev) cudaEventDestroy(s->wave_ev);
  s->wave_side = nullptr;
  s->wave_ev = nullptr;
  s->sub_flow = s->sub_voc = nullptr;
  s->mel = nullptr;
  if (s->stage_in) dc::dev_free(s->stage_in);
  if (s->stage_out) dc::dev_free(s->stage_out);
  s->tails = nullptr;
  s->flow = nullptr;
  s->stage_in = s->stage_out = nullptr;
}

extern "C" dc_status dc_stream_open(dc_model* m, dc_stream** out) {
  if (!m || !out) return DC_ERR_ARG;
  *out = nullptr;
  dc_stream* s = new (std::nothrow) dc_stream();
  if (!s) return DC_ERR_OOM;
  s->model = m;
  cudaError_t e = cudaSuccess;
  dc_status st = DC_OK;
  struct GuardScope {   // every device buffer of a stream gets guard zones when the model asks for them
    bool prev;
    explicit GuardScope(bool on) : prev(dc::g_guard_mode) { dc::g_guard_mode = prev || on; }
    ~GuardScope() { dc::g_guard_mode = prev; }
  } guard_scope((m->cfg.options & DC_OPT_GUARD_ZONES) != 0);
  if (m->sub_flow) {
    st = dc_stream_open(m->sub_flow, &s->sub_flow);
    if (st == DC_OK) st = dc_stream_open(m->sub_voc, &s->sub_voc);
    if (st == DC_OK) e = dc::dev_alloc(&s->mel, (size_t)m->cfg.f_chunk * m->cfg.mel_dim * sizeof(float));
    if (st == DC_OK && e == cudaSuccess && m->cfg.max_wave_frames > 0) {
      // wavefront calls keep a whole call's mel frames on the device and run the vocoder tails on a side stream:
      // both are set up here, so that no decode call allocates or creates anything
      e = dc::dev_alloc(&s->wave_mel, (size_t)m->cfg.max_wave_frames * m->cfg.mel_dim * sizeof(float));
      if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->wave_side, cudaStreamNonBlocking);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->wave_ev, cudaEventDisableTiming);
      if (e == cudaSuccess) s->wave_mel_frames = m->cfg.max_wave_frames;
    }
  } else if (m->flow) {
    st = dc::flow_state_open(m->flow, &s->flow);
  } else {
    s->rng_id = m->streams_opened++;
    for (const F32Layer& L : m->layers) {
      DevBuf b{nullptr, (size_t)L.ring_cap * L.C_in * sizeof(float)};
      e = dc::dev_alloc(&b.p, b.bytes);
      if (e != cudaSuccess) break;
      s->f32_rings.push_back(b);
      e = cudaMemset(b.p, 0, b.bytes);
      if (e != cudaSuccess) break;
    }
    if (e == cudaSuccess) e = dc::dev_alloc(&s->d_call, sizeof(dc::F32Call));
    if (e == cudaSuccess && m->cfg.pipeline == DC_PIPE_VOCODER) {
      e = dc::dev_alloc(&s->tails, 2 * 12 * sizeof(float));
      if (e == cudaSuccess) e = cudaMemset(s->tails, 0, 2 * 12 * sizeof(float));
    }
    if (e == cudaSuccess) {
      dc::F32StreamPtrs hp{};
      for (size_t l = 0; l < s->f32_rings.size() && l < (size_t)dc::F32_MAX_LAYERS; ++l) hp.ring[l] = (float*)s->f32_rings[l].p;
      hp.tails = s->tails;
      e = dc::dev_alloc(&s->d_ptrs, sizeof(hp));
      if (e == cudaSuccess) e = cudaMemcpy(s->d_ptrs, &hp, sizeof(hp), cudaMemcpyHostToDevice);
    }
  }
  if (e == cudaSuccess && st == DC_OK) {
    e = dc::dev_alloc(&s->stage_in, (size_t)(m->cfg.f_chunk + m->cfg.f_lookahead) * m->in_dim * sizeof(float));
    if (e == cudaSuccess) e = dc::dev_alloc(&s->stage_out, (size_t)m->cfg.f_chunk * m->out_per_frame * sizeof(float));
  }
  if (e != cudaSuccess) {
    dc::set_error("stream allocation failed: %s", cudaGetErrorString(e));
    st = e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
  }
  if (st != DC_OK) {
    free_stream_buffers(s);
    delete s;
    return st;
  }
  if (!m->flow && !m->sub_flow) build_f32_graph(s);
  {
    std::lock_guard<std::mutex> lk(m->mu);
    m->all_streams.push_back(s);
  }
  m->open_streams++;
  m->counters[6]++;
  *out = s;
  return DC_OK;
}

extern "C" dc_status dc_stream_reset(dc_stream* s, void* cuda_stream) {
  if (!s || s->closed) return DC_ERR_STATE;
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  if (s->sub_flow) {
    dc_status st = dc_stream_reset(s->sub_flow, cuda_stream);
    if (st == DC_OK) st = dc_stream_reset(s->sub_voc, cuda_stream);
    if (st != DC_OK) return st;
  } else if (s->flow) {
    dc_status st = dc::flow_state_reset(s->model->flow, s->flow, cs);
    if (st != DC_OK) return st;
  } else {
    for (auto& b : s->f32_rings) DC_CUDA(cudaMemsetAsync(b.p, 0, b.bytes, cs));
    if (s->tails) DC_CUDA(cudaMemsetAsync(s->tails, 0, 2 * 12 * sizeof(float), cs));
  }
  s->frames_total = 0;
  s->chunks = 0;
  s->poisoned = false;
  return DC_OK;
}

extern "C" dc_status dc_stream_close(dc_stream* s) {
  if (!s) return DC_ERR_ARG;
  if (s->closed) return DC_ERR_STATE;
  cudaDeviceSynchronize();
  s->closed = true;
  s->model->open_streams--;
  s->model->counters[6]--;
  free_stream_buffers(s);
  return DC_OK;
}

extern "C" dc_status dc_stream_carry_info(const dc_stream* s, uint64_t* out, int max_entries, int* n_entries) {
  if (!s || !out || !n_entries || max_entries < 0) return DC_ERR_ARG;
  if (s->closed) return DC_ERR_STATE;
  std::vector<DevBuf> bufs;
  if (s->sub_flow) {   // the carries of both halves, flow decoder first
    uint64_t tmp[2 * 128];
    for (const dc_stream* sub : {(const dc_stream*)s->sub_flow, (const dc_stream*)s->sub_voc}) {
      int n = 0;
      dc_status st = dc_stream_carry_info(sub, tmp, 128, &n);
      if (st != DC_OK) return st;
      for (int i = 0; i < n && i < 128; ++i) bufs.push_back(DevBuf{(void*)(uintptr_t)tmp[2 * i], (size_t)tmp[2 * i + 1]});
    }
  } else if (s->flow) {
    bufs.resize(64);
    int n = 0;
    dc::flow_state_buffers(s->flow, bufs.data(), 64, &n);
    bufs.resize(n);
  } else {
    bufs = s->f32_rings;
    if (s->tails) bufs.push_back(DevBuf{s->tails, 2 * 12 * sizeof(float)});
  }
  *n_entries = (int)bufs.size();
  for (int i = 0; i < (int)bufs.size() && i < max_entries; ++i) {
    out[2 * i] = (uint64_t)(uintptr_t)bufs[i].p;
    out[2 * i + 1] = (uint64_t)bufs[i].bytes;
  }
  return DC_OK;
}

// ---------------------------------------------------------------------------------------------
// snapshots
// ---------------------------------------------------------------------------------------------

struct dc_snapshot {
  const dc_model* model = nullptr;
  void*     data = nullptr;          // the carry buffers, back to back, in dc_stream_carry_info order
  size_t    bytes = 0;
  long long frames_total = 0, chunks = 0, flow_frames = 0;
  int       rng_id = 0;
  dc_snapshot* sub_flow = nullptr;   // DC_PIPE_TOKEN2WAV: the two halves
  dc_snapshot* sub_voc = nullptr;
};

static std::vector<DevBuf> carry_buffers(const dc_stream* s) {
  std::vector<DevBuf> bufs;
  if (s->flow) {
    bufs.resize(64);
    int n = 0;
    dc::flow_state_buffers(s->flow, bufs.data(), 64, &n);
    bufs.resize((size_t)n);
  } else if (!s->sub_flow) {
    bufs = s->f32_rings;
    if (s->tails) bufs.push_back(DevBuf{s->tails, 2 * 12 * sizeof(float)});
  }
  return bufs;
}

extern "C" dc_status dc_snapshot_free(dc_snapshot* sn) {
  if (!sn) return DC_ERR_ARG;
  if (sn->sub_flow) dc_snapshot_free(sn->sub_flow);
  if (sn->sub_voc) dc_snapshot_free(sn->sub_voc);
  if (sn->data) dc::dev_free(sn->data);
  delete sn;
  return DC_OK;
}

extern "C" dc_status dc_stream_snapshot(dc_stream* s, dc_snapshot** out, void* cuda_stream) {
  if (!s || !out) return DC_ERR_ARG;
  *out = nullptr;
  if (s->closed || s->poisoned) return DC_ERR_STATE;
  dc_snapshot* sn = new (std::nothrow) dc_snapshot();
  if (!sn) return DC_ERR_OOM;
  sn->model = s->model;
  sn->frames_total = s->frames_total;
  sn->chunks = s->chunks;
  dc_status st = DC_OK;
  if (s->sub_flow) {
    st = dc_stream_snapshot(s->sub_flow, &sn->sub_flow, cuda_stream);
    if (st == DC_OK) st = dc_stream_snapshot(s->sub_voc, &sn->sub_voc, cuda_stream);
  } else {
    if (s->flow) {
      sn->flow_frames = dc::flow_state_frames(s->flow);
      sn->rng_id = dc::flow_state_rng_id(s->flow);
    } else {
      sn->rng_id = s->rng_id;
    }
    const std::vector<DevBuf> bufs = carry_buffers(s);
    for (const DevBuf& b : bufs) sn->bytes += b.bytes;
    cudaError_t e = dc::dev_alloc(&sn->data, sn->bytes ? sn->bytes : 1);
    size_t off = 0;
    for (size_t i = 0; i < bufs.size() && e == cudaSuccess; ++i) {
      e = cudaMemcpyAsync((char*)sn->data + off, bufs[i].p, bufs[i].bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream);
      off += bufs[i].bytes;
    }
    if (e != cudaSuccess) {
      dc::set_error("dc_stream_snapshot: %s", cudaGetErrorString(e));
      st = e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
    }
  }
  if (st != DC_OK) {
    dc_snapshot_free(sn);
    return st;
  }
  *out = sn;
  return DC_OK;
}

extern "C" dc_status dc_stream_restore(dc_stream* s, const dc_snapshot* sn, void* cuda_stream) {
  if (!s || !sn) return DC_ERR_ARG;
  if (s->closed || sn->model != s->model) {
    dc::set_error("dc_stream_restore: closed stream, or a snapshot of another model");
    return DC_ERR_STATE;
  }
  if (s->sub_flow) {
    dc_status st = dc_stream_restore(s->sub_flow, sn->sub_flow, cuda_stream);
    if (st == DC_OK) st = dc_stream_restore(s->sub_voc, sn->sub_voc, cuda_stream);
    if (st != DC_OK) return st;
  } else {
    const std::vector<DevBuf> bufs = carry_buffers(s);
    size_t total = 0;
    for (const DevBuf& b : bufs) total += b.bytes;
    if (total != sn->bytes) return DC_ERR_STATE;
    size_t off = 0;
    for (const DevBuf& b : bufs) {   // in place: the carries keep their addresses
      DC_CUDA(cudaMemcpyAsync(b.p, (const char*)sn->data + off, b.bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream));
      off += b.bytes;
    }
    if (s->flow) {
      dc::flow_state_set_frames(s->flow, sn->flow_frames);
      dc::flow_state_set_rng_id(s->flow, sn->rng_id);   // the session keeps its random stream wherever it lives
    } else {
      s->rng_id = sn->rng_id;
    }
  }
  s->frames_total = sn->frames_total;
  s->chunks = sn->chunks;
  s->poisoned = false;
  return DC_OK;
}

// ---------------------------------------------------------------------------------------------
// the chunk step
// ---------------------------------------------------------------------------------------------

// Enqueues the layers of one fp32 chunk step.  With use_call the kernels take the per-call values
// from the model's device-side call record (graph capture); otherwise they get them by value.
static void enqueue_f32(dc_stream* s, bool use_call, const float* feats, int T, float* out, cudaStream_t cs, bool pdl,
                        int* launches) {
  dc_model* m = s->model;
  const int nL = (int)m->layers.size();
  for (int l = 0; l < nL; ++l) {
    const F32Layer& L = m->layers[l];
    const long long pos = s->frames_total * L.rate_in;
    const int Tin = T * L.rate_in;
    const int Tgrid = use_call ? m->cfg.f_chunk * L.rate_in : Tin;
    float* ring = (float*)s->f32_rings[l].p;
    if (L.kind == 2) {
      dc::HeadIstftF32 h{};
      h.in_ring = ring; h.in_mask = L.ring_cap - 1; h.C = L.C_in;
      h.W = m->d_w + L.w_off; h.bias = m->d_w + L.b_off; h.clamp = m->cfg.logmag_clamp;
      if (use_call) {
        h.call = s->d_call; h.rate_in = L.rate_in; h.tails = s->tails;
      } else {
        h.pos = pos; h.T = Tin;
        h.tail_in = s->tails + 12 * (s->chunks & 1);
        h.tail_out = s->tails + 12 * ((s->chunks + 1) & 1);
        h.pcm = out;
      }
      dc::ProfScope ps(&m->prof, 6, cs);
      dc::launch_head_istft_f32(h, cs, Tgrid, pdl);
    } else {
      dc::TapConvF32 p{};
      p.in_ring = ring; p.in_mask = L.ring_cap - 1; p.C_in = L.C_in;
      p.first_layer = l == 0; p.last_layer = l + 1 == nL; p.rate_in = L.rate_in;
      if (use_call) {
        p.call = s->d_call;
      } else {
        p.pos_in = pos; p.T_in = Tin;
        if (l == 0) p.in_direct = feats;
      }
      if (l == 0) { p.save_ring = ring; p.save_rows = L.halo; }
      if (L.kind == 0) {
        p.n_taps = 3; p.shift[0] = 2 * L.dil; p.shift[1] = L.dil; p.shift[2] = 0; p.n_phase = 1;
        p.w_tap_stride = (long long)L.C_in * L.C_out; p.w_phase_stride = 0;
      } else {
        p.n_taps = 2; p.shift[0] = 0; p.shift[1] = 1; p.shift[2] = 0; p.n_phase = L.stride;
        p.w_tap_stride = (long long)L.stride * L.C_in * L.C_out; p.w_phase_stride = (long long)L.C_in * L.C_out;
      }
      p.W = m->d_w + L.w_off; p.bias = m->d_w + L.b_off; p.C_out = L.C_out;
      p.residual_silu = L.residual_silu; p.post_silu = L.post_silu;
      if (L.excite) {
        p.exc_std = m->cfg.excitation_std; p.exc_seed_lo = m->cfg.excitation_seed_lo; p.exc_seed_hi = m->cfg.excitation_seed_hi;
        p.exc_rng_id = s->rng_id;
      }
      if (l + 1 < nL) {
        p.out_ring = (float*)s->f32_rings[l + 1].p; p.out_mask = m->layers[l + 1].ring_cap - 1;
      } else if (!use_call) {
        p.out_direct = out; p.pos_out = pos * p.n_phase;
      }
      dc::ProfScope ps(&m->prof, 5, cs);
      dc::launch_tapconv_f32(p, cs, Tgrid, pdl);
    }
    ++*launches;
  }
}

// Captures the stream's chunk step once (at dc_stream_open): afterwards a chunk is one graph launch.
static void build_f32_graph(dc_stream* s) {
  dc_model* m = s->model;
  if (m->cfg.options & DC_OPT_NO_GRAPH) return;
  cudaStream_t cap = nullptr;
  if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return; }
  // programmatic dependent launch is left off here: measured on the vocoder tail it made the step
  // slower (0.200 ms vs 0.169 ms per chunk), the kernels are too short to gain from early prologues
  const bool pdl = false;
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
    dc::F32Call dummy{};
    dc::launch_set_f32_call(dummy, s->d_call, cap);
    int n = 1;
    enqueue_f32(s, true, nullptr, 0, nullptr, cap, pdl, &n);
    if (cudaStreamEndCapture(cap, &graph) == cudaSuccess && graph != nullptr) {
      size_t n_nodes = 0;
      cudaGraphGetNodes(graph, nullptr, &n_nodes);
      std::vector<cudaGraphNode_t> nodes(n_nodes);
      cudaGraphGetNodes(graph, nodes.data(), &n_nodes);
      for (cudaGraphNode_t nd : nodes) {
        cudaGraphNodeType ty;
        cudaKernelNodeParams kp{};
        if (cudaGraphNodeGetType(nd, &ty) == cudaSuccess && ty == cudaGraphNodeTypeKernel &&
            cudaGraphKernelNodeGetParams(nd, &kp) == cudaSuccess && kp.func == dc::set_f32_call_func())
          s->g_set_node = nd;
      }
      if (s->g_set_node != nullptr && cudaGraphInstantiate(&s->g_exec, graph, 0) == cudaSuccess) {
        s->g_graph = graph;
        s->g_launches = n;
        graph = nullptr;
      } else {
        s->g_exec = nullptr;
      }
    }
  }
  cudaGetLastError();
  if (graph) cudaGraphDestroy(graph);
  cudaStreamDestroy(cap);
}

// The layers of one fp32 chunk step for up to max_batch streams at once: every layer is ONE launch whose grid planes
// are the slots of the batch record (stream, frames, pointers); per slot the tiles, the reduction split and the
// arithmetic are those of the single-stream step, so a stream's bytes do not depend on who shares its launch.
static void enqueue_f32_batch(dc_model* m, cudaStream_t cs, int* launches) {
  const int nL = (int)m->layers.size(), nb = m->cfg.max_batch;
  for (int l = 0; l < nL; ++l) {
    const F32Layer& L = m->layers[l];
    const int Tgrid = m->cfg.f_chunk * L.rate_in;
    if (L.kind == 2) {
      dc::HeadIstftF32 h{};
      h.batch = m->d_batch; h.layer = l; h.rate_in = L.rate_in;
      h.in_mask = L.ring_cap - 1; h.C = L.C_in;
      h.W = m->d_w + L.w_off; h.bias = m->d_w + L.b_off; h.clamp = m->cfg.logmag_clamp;
      dc::ProfScope ps(&m->prof, 6, cs);
      dc::launch_head_istft_f32(h, cs, Tgrid, false, nb);
    } else {
      dc::TapConvF32 p{};
      p.batch = m->d_batch; p.layer = l;
      p.in_mask = L.ring_cap - 1; p.C_in = L.C_in;
      p.first_layer = l == 0; p.last_layer = l + 1 == nL; p.rate_in = L.rate_in;
      if (l == 0) p.save_rows = L.halo;
      if (L.kind == 0) {
        p.n_taps = 3; p.shift[0] = 2 * L.dil; p.shift[1] = L.dil; p.shift[2] = 0; p.n_phase = 1;
        p.w_tap_stride = (long long)L.C_in * L.C_out; p.w_phase_stride = 0;
      } else {
        p.n_taps = 2; p.shift[0] = 0; p.shift[1] = 1; p.shift[2] = 0; p.n_phase = L.stride;
        p.w_tap_stride = (long long)L.stride * L.C_in * L.C_out; p.w_phase_stride = (long long)L.C_in * L.C_out;
      }
      p.W = m->d_w + L.w_off; p.bias = m->d_w + L.b_off; p.C_out = L.C_out;
      p.residual_silu = L.residual_silu; p.post_silu = L.post_silu;
      if (L.excite) {
        p.exc_std = m->cfg.excitation_std; p.exc_seed_lo = m->cfg.excitation_seed_lo; p.exc_seed_hi = m->cfg.excitation_seed_hi;
      }
      if (l + 1 < nL) p.out_mask = m->layers[l + 1].ring_cap - 1;
      dc::ProfScope ps(&m->prof, 5, cs);
      dc::launch_tapconv_f32(p, cs, Tgrid, false, nb);
    }
    ++*launches;
  }
}

// Captured once per model (at dc_create): the batch step is one graph launch, only the slot records change.
static void build_f32_batch_graph(dc_model* m) {
  if (m->cfg.options & DC_OPT_NO_GRAPH) return;
  cudaStream_t cap = nullptr;
  if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return; }
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
    static const dc::F32Batch empty{};
    dc::launch_set_f32_batch(empty, m->d_batch, cap);
    int n = 1;
    enqueue_f32_batch(m, cap, &n);
    if (cudaStreamEndCapture(cap, &graph) == cudaSuccess && graph != nullptr) {
      size_t n_nodes = 0;
      cudaGraphGetNodes(graph, nullptr, &n_nodes);
      std::vector<cudaGraphNode_t> nodes(n_nodes);
      cudaGraphGetNodes(graph, nodes.data(), &n_nodes);
      for (cudaGraphNode_t nd : nodes) {
        cudaGraphNodeType ty;
        cudaKernelNodeParams kp{};
        if (cudaGraphNodeGetType(nd, &ty) == cudaSuccess && ty == cudaGraphNodeTypeKernel &&
            cudaGraphKernelNodeGetParams(nd, &kp) == cudaSuccess && kp.func == dc::set_f32_batch_func())
          m->gb_set_node = nd;
      }
      if (m->gb_set_node != nullptr && cudaGraphInstantiate(&m->gb_exec, graph, 0) == cudaSuccess) {
        m->gb_graph = graph;
        m->gb_launches = n;
        graph = nullptr;
      } else {
        m->gb_exec = nullptr;
      }
    }
  }
  cudaGetLastError();
  if (graph) cudaGraphDestroy(graph);
  cudaStreamDestroy(cap);
}

// One chunk for each of n streams of an fp32 model (admitted by the caller).
static dc_status decode_f32_batch(dc_model* m, int n, dc_stream* const* streams, const float* const* feats, const int* T, float* const* out,
                                  cudaStream_t cs, int* launches) {
  dc::F32Batch hb{};
  hb.n = n;
  for (int i = 0; i < n; ++i) {
    dc_stream* s = streams[i];
    hb.s[i].call = dc::F32Call{s->frames_total, T[i], (int)(s->chunks & 1), feats[i], out[i], s->rng_id};
    hb.s[i].ptrs = s->d_ptrs;
  }
  if (m->gb_exec != nullptr && !m->prof.on) {
    dc::F32Batch* dst = m->d_batch;
    void* args[2] = {&hb, &dst};
    cudaKernelNodeParams kp{};
    kp.func = const_cast<void*>(dc::set_f32_batch_func());
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(dc::F32_MAX_BATCH);
    kp.kernelParams = args;
    DC_CUDA(cudaGraphExecKernelNodeSetParams(m->gb_exec, m->gb_set_node, &kp));
    DC_CUDA(cudaGraphLaunch(m->gb_exec, cs));
    *launches += m->gb_launches;
    m->counters[7]++;
    return DC_OK;
  }
  dc::launch_set_f32_batch(hb, m->d_batch, cs);
  ++*launches;
  enqueue_f32_batch(m, cs, launches);
  DC_CUDA(cudaGetLastError());
  return DC_OK;
}

static dc_status decode_f32(dc_stream* s, const float* feats, int T, float* out, cudaStream_t cs, int* launches) {
  dc_model* m = s->model;
  if (s->g_exec != nullptr && !m->prof.on) {
    dc::F32Call v{s->frames_total, T, (int)(s->chunks & 1), feats, out, s->rng_id};
    dc::F32Call* dst = s->d_call;
    void* args[2] = {&v, &dst};
    cudaKernelNodeParams kp{};
    kp.func = const_cast<void*>(dc::set_f32_call_func());
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(32);
    kp.kernelParams = args;
    DC_CUDA(cudaGraphExecKernelNodeSetParams(s->g_exec, s->g_set_node, &kp));
    DC_CUDA(cudaGraphLaunch(s->g_exec, cs));
    *launches += s->g_launches;
    m->counters[7]++;
    return DC_OK;
  }
  enqueue_f32(s, false, feats, T, out, cs, false, launches);
  DC_CUDA(cudaGetLastError());
  return DC_OK;
}

// The kernels read the caller's chunk and write its output with 16-byte accesses.
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// device_ptrs: feats / out are what the kernels will dereference (device pointers, or the device alias of a
// page-locked host buffer), so they must be 16-byte aligned; host buffers that are staged need no alignment.
static dc_status admit(dc_stream* s, const float* feats, int T, float* out, bool device_ptrs = true) {
  if (!s) return DC_ERR_ARG;
  if (s->closed || s->poisoned) return DC_ERR_STATE;
  if (!feats || !out) {
    s->model->counters[3]++;
    return DC_ERR_ARG;
  }
  if (device_ptrs && (!aligned16(feats) || !aligned16(out))) {
    s->model->counters[3]++;
    dc::set_error("feats (%p) and out (%p) must be 16-byte aligned device pointers", (const void*)feats, (const void*)out);
    return DC_ERR_ARG;
  }
  const int f_call = s->model->cfg.f_chunk + s->model->cfg.f_lookahead;   // committed frames are bounded by f_chunk, presented ones by this
  if (T < 1 || T > f_call) {
    s->model->counters[2]++;
    dc::set_error("n_frames = %d violates 1 <= n_frames <= f_chunk + f_lookahead = %d", T, f_call);
    return DC_ERR_FRAMES;
  }
  return DC_OK;
}

extern "C" dc_status dc_decode_chunk(dc_stream* s, const float* feats, int T, float* out, int* n_out, void* cuda_stream) {
  dc_status st = admit(s, feats, T, out);
  if (st != DC_OK) return st;
  dc_model* m = s->model;
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  int launches = 0;
  if (m->sub_flow) {   // mel frames never leave the device: the flow decoder's output is the vocoder tail's input
    st = dc_decode_chunk(s->sub_flow, feats, T, s->mel, nullptr, cuda_stream);
    if (st == DC_OK) st = dc_decode_chunk(s->sub_voc, s->mel, T < m->cfg.f_chunk ? T : m->cfg.f_chunk, out, nullptr, cuda_stream);
  } else if (m->flow) {
    st = dc::flow_decode(m->flow, 1, &s->flow, &feats, &T, &out, cs, &launches);
  } else {
    st = decode_f32(s, feats, T, out, cs, &launches);
  }
  m->counters[5] += (uint64_t)launches;
  if (st != DC_OK) {
    s->poisoned = true;
    return st;
  }
  const int Tc = T < m->cfg.f_chunk ? T : m->cfg.f_chunk;   // frames beyond f_chunk were look-ahead: attended, not committed
  s->frames_total += Tc;
  s->chunks += 1;
  m->counters[0] += 1;
  m->counters[1] += (uint64_t)Tc;
  if (n_out) *n_out = Tc * m->out_per_frame;
  return DC_OK;
}

namespace {
// Host-side hook of the composite's wavefront: as soon as the pass that finishes chunk j of a stream is
// enqueued, the vocoder tail of that chunk is enqueued on the stream's side stream behind an event, so that it
// runs beside the flow decoder's next passes (which leave most SMs idle) instead of after them.
struct WaveTail {
  dc_stream* const* streams;
  cudaStream_t      main_st;
  bool              side;          // false while profiling: everything on the caller's stream
  float* const*     out;
  const long long*  n_frames;
  dc_status         st = DC_OK;
};

void wave_tail_chunk(void* ctx, int i, long long j) {
  WaveTail* w = static_cast<WaveTail*>(ctx);
  if (w->st != DC_OK) return;
  dc_stream* s = w->streams[i];
  dc_model* m = s->model;
  const int fc = m->cfg.f_chunk;
  const int T = (int)(w->n_frames[i] - j * fc < fc ? w->n_frames[i] - j * fc : fc);
  cudaStream_t ts = w->side ? s->wave_side : w->main_st;
  if (w->side && (cudaEventRecord(s->wave_ev, w->main_st) != cudaSuccess || cudaStreamWaitEvent(ts, s->wave_ev, 0) != cudaSuccess)) {
    w->st = DC_ERR_CUDA;
    return;
  }
  w->st = dc_decode_chunk(s->sub_voc, s->wave_mel + j * fc * m->cfg.mel_dim, T, w->out[i] + j * fc * m->out_per_frame, nullptr, (void*)ts);
}
}  // namespace

extern "C" dc_status dc_decode_wavefront_batch(dc_model* m, int n, dc_stream* const* streams, const float* const* feats,
                                               const long long* n_frames, float* const* out, void* cuda_stream) {
  if (!m || !streams || !feats || !n_frames || !out) return DC_ERR_ARG;
  if (!m->flow && !m->sub_flow) {
    dc::set_error("wavefront decoding serves the flow and token2wav pipelines only");
    return DC_ERR_CONFIG;
  }
  if (n < 1 || (long long)n * m->cfg.n_steps > m->cfg.max_batch) {
    m->counters[3]++;
    dc::set_error("wavefront decoding keeps n_steps = %d chunks per stream in flight: %d streams need max_batch >= %d", m->cfg.n_steps, n,
                  n * m->cfg.n_steps);
    return DC_ERR_ARG;
  }
  for (int i = 0; i < n; ++i) {
    dc_stream* s = streams[i];
    if (!s) return DC_ERR_ARG;
    if (s->closed || s->poisoned || s->model != m) return DC_ERR_STATE;
    if (!feats[i] || !out[i] || n_frames[i] < 1) {
      m->counters[3]++;
      return DC_ERR_ARG;
    }
    if (!aligned16(feats[i]) || !aligned16(out[i])) {
      m->counters[3]++;
      dc::set_error("feats[%d] (%p) and out[%d] (%p) must be 16-byte aligned device pointers", i, (const void*)feats[i], i, (const void*)out[i]);
      return DC_ERR_ARG;
    }
    if (m->sub_flow && n_frames[i] > s->wave_mel_frames) {
      m->counters[3]++;
      dc::set_error("wavefront call of %lld frames on a token2wav stream opened with max_wave_frames = %lld", n_frames[i], s->wave_mel_frames);
      return DC_ERR_ARG;
    }
    for (int j = 0; j < i; ++j)
      if (streams[j] == s) {
        m->counters[3]++;
        dc::set_error("stream %d appears twice in the batch", i);
        return DC_ERR_ARG;
      }
  }
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  const int fc = m->cfg.f_chunk;
  dc_model* fm = m->sub_flow ? m->sub_flow : m;
  std::vector<dc::FlowState*> states((size_t)n);
  std::vector<float*> mels((size_t)n);
  for (int i = 0; i < n; ++i) states[(size_t)i] = m->sub_flow ? streams[i]->sub_flow->flow : streams[i]->flow;
  dc_status st = DC_OK;
  int launches = 0;
  if (m->sub_flow) {
    // each stream's mel frames stay on the device, in a buffer of the stream; its vocoder tails run on a
    // CUDA stream of its own
    for (int i = 0; i < n; ++i) {
      dc_stream* s = streams[i];
      mels[(size_t)i] = s->wave_mel;
    }
    WaveTail w{streams, cs, !(m->sub_voc->prof.on || m->sub_flow->prof.on), out, n_frames};
    st = dc::flow_decode_wave(fm->flow, n, states.data(), feats, fm->in_dim, n_frames, mels.data(), cs, &launches, wave_tail_chunk, &w);
    if (st == DC_OK) st = w.st;
    for (int i = 0; i < n && st == DC_OK && w.side; ++i)   // the caller's stream continues only after every stream's last tail
      if (cudaEventRecord(streams[i]->wave_ev, streams[i]->wave_side) != cudaSuccess ||
          cudaStreamWaitEvent(cs, streams[i]->wave_ev, 0) != cudaSuccess)
        st = DC_ERR_CUDA;
  } else {
    st = dc::flow_decode_wave(fm->flow, n, states.data(), feats, fm->in_dim, n_frames, out, cs, &launches, nullptr, nullptr);
  }
  fm->counters[5] += (uint64_t)launches;
  if (st == DC_ERR_ARG) {   // refused before anything ran: the streams are untouched
    m->counters[3]++;
    return st;
  }
  if (st != DC_OK) {
    for (int i = 0; i < n; ++i) {
      streams[i]->poisoned = true;
      if (m->sub_flow) streams[i]->sub_flow->poisoned = true;
    }
    return st;
  }
  for (int i = 0; i < n; ++i) {
    const long long n_chunks = (n_frames[i] + fc - 1) / fc;
    for (dc_stream* s : {streams[i], m->sub_flow ? streams[i]->sub_flow : (dc_stream*)nullptr}) {
      if (!s) continue;
      s->frames_total += n_frames[i];
      s->chunks += n_chunks;
      s->model->counters[0] += (uint64_t)n_chunks;
      s->model->counters[1] += (uint64_t)n_frames[i];
    }
  }
  return DC_OK;
}

extern "C" dc_status dc_decode_wavefront(dc_stream* s, const float* feats, long long n_frames, float* out, long long* n_out,
                                         void* cuda_stream) {
  if (!s) return DC_ERR_ARG;
  if (s->closed || s->poisoned) return DC_ERR_STATE;
  dc_status st = dc_decode_wavefront_batch(s->model, 1, &s, &feats, &n_frames, &out, cuda_stream);
  if (st == DC_OK && n_out) *n_out = n_frames * s->model->out_per_frame;
  return st;
}

extern "C" dc_status dc_decode_batch(dc_model* m, int n, dc_stream* const* streams, const float* const* feats,
                                     const int* n_frames, float* const* out, void* cuda_stream) {
  if (!m || !streams || !feats || !n_frames || !out) return DC_ERR_ARG;
  if (n < 1 || n > m->cfg.max_batch) {
    m->counters[3]++;
    dc::set_error("batch of %d streams, max_batch = %d", n, m->cfg.max_batch);
    return DC_ERR_ARG;
  }
  std::vector<dc::FlowState*> states((size_t)n);
  for (int i = 0; i < n; ++i) {
    dc_status st = admit(streams[i], feats[i], n_frames[i], out[i]);
    if (st != DC_OK) return st;
    if (streams[i]->model != m) {
      m->counters[3]++;
      return DC_ERR_STATE;
    }
    for (int j = 0; j < i; ++j)
      if (streams[j] == streams[i]) {
        m->counters[3]++;
        dc::set_error("stream %d appears twice in the batch", i);
        return DC_ERR_ARG;
      }
    states[(size_t)i] = streams[i]->flow;
  }
  int launches = 0;
  dc_status st = DC_OK;
  if (m->sub_flow) {   // flow decoder batched over the streams, then every stream's vocoder tail
    std::vector<dc_stream*> fs((size_t)n);
    std::vector<float*> mels((size_t)n);
    for (int i = 0; i < n; ++i) {
      fs[(size_t)i] = streams[i]->sub_flow;
      mels[(size_t)i] = streams[i]->mel;
    }
    st = dc_decode_batch(m->sub_flow, n, fs.data(), feats, n_frames, mels.data(), cuda_stream);
    // ... then the vocoder tails of all the streams, every layer one launch over the batch (n = 1, or
    // DC_OPT_SERIAL_TAILS: stream by stream, one captured step each)
    if (st == DC_OK) {
      std::vector<dc_stream*> vs((size_t)n);
      std::vector<int> tc((size_t)n);
      for (int i = 0; i < n; ++i) {
        vs[(size_t)i] = streams[i]->sub_voc;
        tc[(size_t)i] = n_frames[i] < m->cfg.f_chunk ? n_frames[i] : m->cfg.f_chunk;
      }
      if (n >= 2 && !(m->cfg.options & DC_OPT_SERIAL_TAILS)) {
        st = dc_decode_batch(m->sub_voc, n, vs.data(), mels.data(), tc.data(), out, cuda_stream);
      } else {
        for (int i = 0; i < n && st == DC_OK; ++i) st = dc_decode_chunk(vs[(size_t)i], mels[(size_t)i], tc[(size_t)i], out[i], nullptr, cuda_stream);
      }
    }
  } else if (m->flow) {
    st = dc::flow_decode(m->flow, n, states.data(), feats, n_frames, out, (cudaStream_t)cuda_stream, &launches);
  } else if (m->d_batch == nullptr) {   // an fp32 model created with max_batch = 1
    st = decode_f32(streams[0], feats[0], n_frames[0], out[0], (cudaStream_t)cuda_stream, &launches);
  } else {
    st = decode_f32_batch(m, n, streams, feats, n_frames, out, (cudaStream_t)cuda_stream, &launches);
  }
  m->counters[5] += (uint64_t)launches;
  if (st != DC_OK) {
    for (int i = 0; i < n; ++i) streams[i]->poisoned = true;
    return st;
  }
  for (int i = 0; i < n; ++i) {
    const int Tc = n_frames[i] < m->cfg.f_chunk ? n_frames[i] : m->cfg.f_chunk;
    streams[i]->frames_total += Tc;
    streams[i]->chunks += 1;
    m->counters[1] += (uint64_t)Tc;
  }
  m->counters[0] += (uint64_t)n;
  return DC_OK;
}

extern "C" dc_status dc_decode_chunk_host(dc_stream* s, const float* feats_host, int T, float* out_host, int* n_out,
                                          void* cuda_stream) {
  dc_status st = admit(s, feats_host, T, out_host, false);
  if (st != DC_OK) return st;
  dc_model* m = s->model;
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  // flow pipeline: page-locked, 16-byte aligned caller buffers are read / written by the kernels themselves
  // (see dc_decode_batch_host); any other buffer is staged
  const float* fin = s->stage_in;
  float* fout = s->stage_out;
  if (m->flow && m->zero_copy) {
    cudaPointerAttributes a{};
    if (cudaPointerGetAttributes(&a, feats_host) == cudaSuccess && a.type == cudaMemoryTypeHost && a.devicePointer != nullptr &&
        aligned16(a.devicePointer))
      fin = static_cast<const float*>(a.devicePointer);
    if (cudaPointerGetAttributes(&a, out_host) == cudaSuccess && a.type == cudaMemoryTypeHost && a.devicePointer != nullptr &&
        aligned16(a.devicePointer))
      fout = static_cast<float*>(a.devicePointer);
    cudaGetLastError();
  }
  if (fin == s->stage_in)
    DC_CUDA(cudaMemcpyAsync(s->stage_in, feats_host, (size_t)T * m->in_dim * sizeof(float), cudaMemcpyHostToDevice, cs));
  int n = 0;
  st = dc_decode_chunk(s, fin, T, fout, &n, cuda_stream);
  if (st != DC_OK) return st;
  if (fout == s->stage_out) DC_CUDA(cudaMemcpyAsync(out_host, s->stage_out, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, cs));
  dc_model* fmod = m->flow ? m : m->sub_flow;   // the model that owns the flow decoder, if any
  if (fmod && fmod->h_err) DC_CUDA(cudaMemcpyAsync(fmod->h_err, dc::flow_error_word(fmod->flow), sizeof(int), cudaMemcpyDeviceToHost, cs));
  DC_CUDA(cudaStreamSynchronize(cs));
  if (fmod && fmod->h_err && *fmod->h_err != 0) {   // a bounded device-side wait gave up: the chunk's result is not valid
    const int code = dc::flow_take_device_error(fmod->flow);   // reads and clears the word
    m->counters[4]++;
    s->poisoned = true;
    dc::set_error("device-side wait timed out (code %d)", code);
    return DC_ERR_TIMEOUT;
  }
  if (n_out) *n_out = n;
  return DC_OK;
}

extern "C" dc_status dc_decode_batch_host(dc_model* m, int n, dc_stream* const* streams, const float* const* feats_host,
                                          const int* n_frames, float* const* out_host, void* cuda_stream) {
  if (!m || !streams || !feats_host || !n_frames || !out_host) return DC_ERR_ARG;
  if (!m->h_in) {
    dc::set_error("dc_decode_batch_host: the model has no staging buffers");
    return DC_ERR_CONFIG;
  }
  if (n < 1 || n > m->cfg.max_batch) return DC_ERR_ARG;
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  dc_model* fmod = m->flow ? m : m->sub_flow;   // the model that owns a flow decoder (and its device error word), if any
  const size_t in_stride = (size_t)(m->cfg.f_chunk + m->cfg.f_lookahead) * m->in_dim, out_stride = (size_t)m->cfg.f_chunk * m->out_per_frame;
  std::vector<const float*> fin((size_t)n);
  std::vector<float*> fout((size_t)n);
  for (int i = 0; i < n; ++i) {
    dc_status st = admit(streams[i], feats_host[i], n_frames[i], out_host[i], false);
    if (st != DC_OK) return st;
    fin[(size_t)i] = m->d_in + (size_t)i * in_stride;
    fout[(size_t)i] = m->d_out + (size_t)i * out_stride;
  }
  // Page-locked caller buffers are read and written by the kernels themselves (the input-preparation kernel
  // pulls the chunks over the bus, the last output-projection epilogue pushes the mel rows back): no staging
  // copy and no copy-engine operation on either side.  Pageable buffers go through one pinned bounce buffer
  // each way: two transfers per step instead of two per stream.
  // (flow pipeline only: its kernels are the ones that can address host memory)
  bool in_direct = m->flow && m->zero_copy, out_direct = m->flow && m->zero_copy;
  for (int i = 0; i < n && (in_direct || out_direct); ++i) {
    cudaPointerAttributes a{};
    if (in_direct) {
      if (cudaPointerGetAttributes(&a, feats_host[i]) == cudaSuccess && a.type == cudaMemoryTypeHost && a.devicePointer != nullptr &&
          aligned16(a.devicePointer)) {
        fin[(size_t)i] = static_cast<const float*>(a.devicePointer);
      } else {
        in_direct = false;
      }
    }
    if (out_direct) {
      if (cudaPointerGetAttributes(&a, out_host[i]) == cudaSuccess && a.type == cudaMemoryTypeHost && a.devicePointer != nullptr &&
          aligned16(a.devicePointer)) {
        fout[(size_t)i] = static_cast<float*>(a.devicePointer);
      } else {
        out_direct = false;
      }
    }
  }
  cudaGetLastError();
  if (!in_direct) {
    for (int i = 0; i < n; ++i) {
      fin[(size_t)i] = m->d_in + (size_t)i * in_stride;
      memcpy(m->h_in + (size_t)i * in_stride, feats_host[i], (size_t)n_frames[i] * m->in_dim * sizeof(float));
    }
    DC_CUDA(cudaMemcpyAsync(m->d_in, m->h_in, (size_t)n * in_stride * sizeof(float), cudaMemcpyHostToDevice, cs));
  }
  if (!out_direct)
    for (int i = 0; i < n; ++i) fout[(size_t)i] = m->d_out + (size_t)i * out_stride;
  dc_status st = dc_decode_batch(m, n, streams, fin.data(), n_frames, fout.data(), cuda_stream);
  if (st != DC_OK) return st;
  if (!out_direct) DC_CUDA(cudaMemcpyAsync(m->h_out, m->d_out, (size_t)n * out_stride * sizeof(float), cudaMemcpyDeviceToHost, cs));
  if (fmod) DC_CUDA(cudaMemcpyAsync(fmod->h_err, dc::flow_error_word(fmod->flow), sizeof(int), cudaMemcpyDeviceToHost, cs));
  DC_CUDA(cudaStreamSynchronize(cs));
  if (fmod && *fmod->h_err != 0) {   // a bounded device-side wait gave up: the results are not valid
    const int code = *fmod->h_err;
    dc::flow_take_device_error(fmod->flow);
    m->counters[4]++;
    for (int i = 0; i < n; ++i) streams[i]->poisoned = true;
    dc::set_error("device-side wait timed out (code %d)", code);
    return DC_ERR_TIMEOUT;
  }
  if (!out_direct)
    for (int i = 0; i < n; ++i)
      memcpy(out_host[i], m->h_out + (size_t)i * out_stride,
             (size_t)(n_frames[i] < m->cfg.f_chunk ? n_frames[i] : m->cfg.f_chunk) * m->out_per_frame * sizeof(float));
  return DC_OK;
}

extern "C" dc_status dc_profile_begin(dc_model* m, int max_launches) {
  if (!m || max_launches < 1 || max_launches > (1 << 20)) return DC_ERR_ARG;
  if (m->sub_flow) {
    dc_status st = dc_profile_begin(m->sub_flow, max_launches);
    return st == DC_OK ? dc_profile_begin(m->sub_voc, max_launches) : st;
  }
  dc::Profiler& p = m->prof;
  if (p.on) return DC_ERR_STATE;
  p.ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_launches];
  p.cls = new (std::nothrow) int[(size_t)max_launches];
  if (!p.ev || !p.cls) return DC_ERR_OOM;
  for (int i = 0; i < 2 * max_launches; ++i) DC_CUDA(cudaEventCreate(&p.ev[i]));
  p.cap = max_launches;
  p.used = 0;
  p.on = true;
  if (m->flow) dc::flow_set_profiler(m->flow, &p);
  return DC_OK;
}

extern "C" dc_status dc_profile_end(dc_model* m, double ms[8], uint64_t launches[8]) {
  if (!m || !ms || !launches) return DC_ERR_ARG;
  if (m->sub_flow) {   // the two halves use disjoint kernel classes
    double ms2[8];
    uint64_t l2[8];
    dc_status st = dc_profile_end(m->sub_flow, ms, launches);
    if (st == DC_OK) st = dc_profile_end(m->sub_voc, ms2, l2);
    for (int i = 0; i < 8 && st == DC_OK; ++i) { ms[i] += ms2[i]; launches[i] += l2[i]; }
    return st;
  }
  dc::Profiler& p = m->prof;
  if (!p.on) return DC_ERR_STATE;
  p.on = false;
  if (m->flow) dc::flow_set_profiler(m->flow, nullptr);
  DC_CUDA(cudaDeviceSynchronize());
  for (int i = 0; i < 8; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (int i = 0; i < p.used; ++i) {
    float t = 0.f;
    DC_CUDA(cudaEventElapsedTime(&t, p.ev[2 * i], p.ev[2 * i + 1]));
    ms[p.cls[i] & 7] += (double)t;
    launches[p.cls[i] & 7] += 1;
  }
  for (int i = 0; i < 2 * p.cap; ++i) cudaEventDestroy(p.ev[i]);
  delete[] p.ev;
  delete[] p.cls;
  p.ev = nullptr; p.cls = nullptr; p.cap = p.used = 0;
  return DC_OK;
}

extern "C" dc_status dc_get_counters(const dc_model* m, uint64_t counters[8]) {
  if (!m || !counters) return DC_ERR_ARG;
  if (m->flow) {   // synchronous read of the device error word (asynchronous decode calls cannot see it)
    const int code = dc::flow_take_device_error(m->flow);
    if (code > 0) const_cast<dc_model*>(m)->counters[4]++;
  }
  for (int i = 0; i < 8; ++i) counters[i] = m->counters[i].load();
  if (m->flow) counters[7] += dc::flow_graph_launches(m->flow);
  if (m->sub_flow) {   // kernel launches, graph launches and device time-outs are counted where they happen
    uint64_t a[8], b[8];
    dc_get_counters(m->sub_flow, a);
    dc_get_counters(m->sub_voc, b);
    counters[4] += a[4] + b[4];
    counters[5] += a[5] + b[5];
    counters[7] += a[7] + b[7];
  }
  return DC_OK;
}

extern "C" dc_status dc_stream_check_guards(dc_stream* s, int* n_damaged) {
  if (!s) return DC_ERR_ARG;
  if (s->closed) return DC_ERR_STATE;
  if (n_damaged) *n_damaged = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return DC_ERR_CUDA;
  int total = 0;
  std::vector<dc_stream*> parts = {s};
  if (s->sub_flow) parts.push_back(s->sub_flow);
  if (s->sub_voc) parts.push_back(s->sub_voc);
  for (dc_stream* q : parts) {
    std::vector<const void*> bufs;
    for (const DevBuf& b : carry_buffers(q)) bufs.push_back(b.p);
    for (const void* extra : {(const void*)q->mel, (const void*)q->wave_mel, (const void*)q->stage_in, (const void*)q->stage_out,
                              (const void*)q->d_call, (const void*)q->d_ptrs})
      if (extra) bufs.push_back(extra);
    for (const void* b : bufs) {
      const int bad = dc::damaged_guards(b);
      if (bad < 0) return DC_ERR_CUDA;
      total += bad;
    }
  }
  if (n_damaged) *n_damaged = total;
  if (total > 0) {
    dc::set_error("%d guard zone(s) around the stream's device buffers were overwritten", total);
    return DC_ERR_STATE;
  }
  return DC_OK;
}

extern "C" dc_status dc_measure_fp32_peak(double* tflops) {
  if (!tflops) return DC_ERR_ARG;
  *tflops = 0.0;
  cudaError_t e = dc::measure_fp32_peak(tflops);
  if (e != cudaSuccess) {
    dc::set_error("dc_measure_fp32_peak: %s", cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
  }
  return DC_OK;
}

extern "C" dc_status dc_test_fail_allocation(int nth) {
  if (nth < 0) return DC_ERR_ARG;
  dc::g_fail_countdown = nth;
  return DC_OK;
}

extern "C" dc_status dc_selftest_bounded_wait(int max_polls) { return dc::flow_selftest_bounded_wait(max_polls); }

extern "C" const char* dc_status_str(dc_status s) {
  switch (s) {
    case DC_OK: return "DC_OK";
    case DC_ERR_ARG: return "DC_ERR_ARG";
    case DC_ERR_CONFIG: return "DC_ERR_CONFIG";
    case DC_ERR_FRAMES: return "DC_ERR_FRAMES";
    case DC_ERR_OOM: return "DC_ERR_OOM";
    case DC_ERR_CUDA: return "DC_ERR_CUDA";
    case DC_ERR_TIMEOUT: return "DC_ERR_TIMEOUT";
    case DC_ERR_STATE: return "DC_ERR_STATE";
  }
  return "DC_ERR_UNKNOWN";
}

extern "C" const char* dc_last_error(void) { return dc::g_last_error.c_str(); }
