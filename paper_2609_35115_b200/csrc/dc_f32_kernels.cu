// fp32 kernels of the conv pipeline and the vocoder tail: a tiled FFMA "tap GEMM" over ring
// buffers (causal conv k=3 with dilation, and the phases of the causal transposed conv), and the
// fused head conv + inverse STFT + overlap-add kernel.  fp32 parity (max err <= 1e-4 of RMS) rules
// out single-pass TF32, so these run on the FP32 pipe.
#include "dc_internal.h"

#include <math.h>

#include <mutex>

namespace dc {

namespace {

constexpr int BM = 64;   // frames per CTA tile
constexpr int BN = 64;   // output channels per CTA tile
constexpr int BK = 16;   // reduction slice
constexpr int NT = 256;  // threads: 16 x 16, each a 4 x 4 micro tile

__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + expf(-z)); }

__device__ __forceinline__ const float* in_row_ptr(const TapConvF32& p, long long t) {
  if (p.in_direct != nullptr && t >= p.pos_in) return p.in_direct + (t - p.pos_in) * p.C_in;
  return p.in_ring + (long long)((int)(t & (long long)p.in_mask)) * p.C_in;
}

__global__ void __launch_bounds__(NT) tapconv_f32_kernel(const TapConvF32 p) {
  __shared__ __align__(16) float As[2][BK][BM + 4];
  __shared__ __align__(16) float Bs[2][BK][BN];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN, phase = blockIdx.z;

  const int a_row = tid >> 2, a_k = (tid & 3) * 4;     // A tile: 64 rows x 16 k, one float4 per thread
  const int b_k = tid >> 4, b_n = (tid & 15) * 4;      // B tile: 16 k x 64 n
  const bool a_ok = (m0 + a_row) < p.T_in;
  const long long t_row = p.pos_in + m0 + a_row;
  const float* Wp = p.W + (long long)phase * p.w_phase_stride;

  const int kb_per_tap = (p.C_in + BK - 1) / BK;
  const int nkb = p.n_taps * kb_per_tap;

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  float4 ra, rb;
  auto gload = [&](int kb) {
    const int tap = kb / kb_per_tap;
    const int c0 = (kb - tap * kb_per_tap) * BK;
    ra = make_float4(0.f, 0.f, 0.f, 0.f);
    rb = ra;
    if (a_ok && c0 + a_k < p.C_in)
      ra = *reinterpret_cast<const float4*>(in_row_ptr(p, t_row - p.shift[tap]) + c0 + a_k);
    if (c0 + b_k < p.C_in && n0 + b_n < p.C_out)
      rb = *reinterpret_cast<const float4*>(Wp + (long long)tap * p.w_tap_stride +
                                            (long long)(c0 + b_k) * p.C_out + n0 + b_n);
  };
  auto sstore = [&](int buf) {
    As[buf][a_k + 0][a_row] = ra.x;
    As[buf][a_k + 1][a_row] = ra.y;
    As[buf][a_k + 2][a_row] = ra.z;
    As[buf][a_k + 3][a_row] = ra.w;
    *reinterpret_cast<float4*>(&Bs[buf][b_k][b_n]) = rb;
  };

  gload(0);
  sstore(0);
  __syncthreads();
  for (int kb = 0; kb < nkb; ++kb) {
    const int cur = kb & 1;
    if (kb + 1 < nkb) gload(kb + 1);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w};
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (kb + 1 < nkb) {
      sstore(cur ^ 1);
      __syncthreads();
    }
  }

  const int n = n0 + tx * 4;
  if (n < p.C_out) {
    const float4 bias = *reinterpret_cast<const float4*>(p.bias + n);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = m0 + ty * 4 + i;
      if (row >= p.T_in) continue;
      const long long t_in = p.pos_in + row;
      float4 v = make_float4(acc[i][0] + bias.x, acc[i][1] + bias.y, acc[i][2] + bias.z, acc[i][3] + bias.w);
      if (p.residual_silu) {
        const float4 x = *reinterpret_cast<const float4*>(in_row_ptr(p, t_in) + n);
        v = make_float4(x.x + silu_f(v.x), x.y + silu_f(v.y), x.z + silu_f(v.z), x.w + silu_f(v.w));
      }
      if (p.post_silu) v = make_float4(silu_f(v.x), silu_f(v.y), silu_f(v.z), silu_f(v.w));
      const long long t_out = (long long)p.n_phase * t_in + phase;
      float* dst = (p.out_direct != nullptr)
                       ? p.out_direct + (t_out - p.pos_out) * p.C_out + n
                       : p.out_ring + (long long)((int)(t_out & (long long)p.out_mask)) * p.C_out + n;
      *reinterpret_cast<float4*>(dst) = v;
    }
  }

  // Carry update of the first layer: its left context for the next chunk is the tail of the
  // caller's chunk, written into ring rows that no CTA of this launch reads (distinct logical
  // frames map to distinct rows because the ring holds f_chunk + halo frames).
  if (p.save_ring != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
    const int first = p.T_in > p.save_rows ? p.T_in - p.save_rows : 0;
    const int c4 = p.C_in >> 2;
    for (int i = tid; i < (p.T_in - first) * c4; i += NT) {
      const int r = first + i / c4, c = (i - (i / c4) * c4) * 4;
      const float4 v = *reinterpret_cast<const float4*>(p.in_direct + (long long)r * p.C_in + c);
      *reinterpret_cast<float4*>(p.save_ring + (long long)((int)((p.pos_in + r) & (long long)p.in_mask)) * p.C_in + c) = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------

constexpr int HT = 64;          // threads per CTA of the head kernel
constexpr int HF = HT - 3;      // new frames per CTA; the first 3 threads recompute the overlap
constexpr int NFFT = 16, NB = 9, NH = 18, HOP = 4, TAIL = NFFT - HOP;

__constant__ float c_cos16[16];  // cos(2 pi j / 16)
__constant__ float c_sin16[16];
__constant__ float c_hann16[16];

__global__ void __launch_bounds__(HT) head_istft_f32_kernel(const HeadIstftF32 p) {
  extern __shared__ __align__(16) float smem[];
  float* Ws = smem;                              // [3*C][NH]
  float* g = smem + 3 * p.C * NH;                // [HT][NFFT] windowed frame signals
  const int tid = threadIdx.x;
  for (int i = tid; i < 3 * p.C * NH; i += HT) Ws[i] = p.W[i];
  __syncthreads();

  const int f_local = blockIdx.x * HF + tid - 3;  // frame index within the chunk (may be < 0)
  const bool is_new = tid >= 3 && f_local < p.T;
  const bool compute = f_local >= 0 && f_local < p.T;   // frames of earlier chunks come from the tail
  float gv[NFFT];
#pragma unroll
  for (int k = 0; k < NFFT; ++k) gv[k] = 0.f;
  if (compute) {
    float z[NH];
#pragma unroll
    for (int o = 0; o < NH; ++o) z[o] = p.bias[o];
    const long long t = p.pos + f_local;
    for (int tap = 0; tap < 3; ++tap) {
      const float* x = p.in_ring + (long long)((int)((t - (2 - tap)) & (long long)p.in_mask)) * p.C;
      const float* w = Ws + tap * p.C * NH;
      for (int c = 0; c < p.C; c += 4) {
        const float4 xv = *reinterpret_cast<const float4*>(x + c);
        const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int o = 0; o < NH; ++o) z[o] = fmaf(xs[q], w[(c + q) * NH + o], z[o]);
      }
    }
    float re[NB], im[NB];
#pragma unroll
    for (int f = 0; f < NB; ++f) {
      const float mag = expf(fminf(z[f], p.clamp));
      float s, c;
      sincosf(z[NB + f], &s, &c);
      re[f] = mag * c;
      im[f] = mag * s;
    }
#pragma unroll
    for (int k = 0; k < NFFT; ++k) {
      float a = re[0] + ((k & 1) ? -re[NB - 1] : re[NB - 1]);
#pragma unroll
      for (int f = 1; f < NB - 1; ++f) {
        const int j = (f * k) & 15;
        a += 2.0f * (re[f] * c_cos16[j] - im[f] * c_sin16[j]);
      }
      gv[k] = c_hann16[k] * a * (1.0f / NFFT);
    }
  }
#pragma unroll
  for (int k = 0; k < NFFT; ++k) g[tid * NFFT + k] = gv[k];
  __syncthreads();

  if (is_new) {
    const float inv_norm = 1.0f / 1.5f;   // sum of the four overlapping squared Hann windows
    float out[HOP];
#pragma unroll
    for (int j = 0; j < HOP; ++j) {
      // sample 4 f + j: contributions of frames f, f-1, f-2, f-3 at offsets j, 4+j, 8+j, 12+j;
      // the part that frames of earlier chunks contribute is the carried tail
      float a = (f_local < 3 && 4 * f_local + j < TAIL) ? p.tail_in[4 * f_local + j] : 0.f;
#pragma unroll
      for (int i = 3; i >= 0; --i) a += g[(tid - i) * NFFT + 4 * i + j];
      out[j] = a * inv_norm;
    }
    *reinterpret_cast<float4*>(p.pcm + 4ll * f_local) = make_float4(out[0], out[1], out[2], out[3]);
    if (f_local == p.T - 1) {
      // tail for the next chunk: samples 4T + q, q in [0,12), from the last three frames
      for (int q = 0; q < TAIL; ++q) {
        float a = 0.f;
        for (int i = 2; i >= 0; --i)
          if (4 * (i + 1) + q < NFFT) a += g[(tid - i) * NFFT + 4 * (i + 1) + q];
        p.tail_out[q] = a;
      }
    }
  }
}

}  // namespace

void launch_tapconv_f32(const TapConvF32& p, cudaStream_t st) {
  dim3 grid((p.T_in + BM - 1) / BM, (p.C_out + BN - 1) / BN, p.n_phase);
  tapconv_f32_kernel<<<grid, NT, 0, st>>>(p);
}

cudaError_t prepare_f32_constants() {
  float c[16], s[16], w[16];
  for (int j = 0; j < 16; ++j) {
    const double a = 2.0 * 3.14159265358979323846 * j / 16.0;
    c[j] = (float)cos(a);
    s[j] = (float)sin(a);
    w[j] = (float)(0.5 - 0.5 * cos(a));
  }
  cudaError_t e = cudaMemcpyToSymbol(c_cos16, c, sizeof(c));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(c_sin16, s, sizeof(s));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(c_hann16, w, sizeof(w));
  return e;
}

void launch_head_istft_f32(const HeadIstftF32& p, cudaStream_t st) {
  const size_t smem = (size_t)(3 * p.C * NH + HT * NFFT) * sizeof(float);
  const int grid = (p.T + HF - 1) / HF;
  head_istft_f32_kernel<<<grid, HT, smem, st>>>(p);
}

}  // namespace dc

// ---------------------------------------------------------------------------------------------
// Allocation-free conv stack (see dc.h).  The activations between blocks live in this array,
// which is part of the library image.  In host code `g_noalloc_scratch` is only a handle for the
// runtime's symbol lookup, never an address to hand to a kernel; the device address comes from
// cudaGetSymbolAddress, once per device.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) float g_noalloc_scratch[DC_NOALLOC_SCRATCH_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
float*     g_noalloc_ptr[kMaxDevices] = {nullptr};
std::mutex g_noalloc_mu;

// Device address of the scratch array on the current device (looked up on first use).
dc_status noalloc_scratch(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    dc::set_error("dc_conv_stack_noalloc: cannot identify the current device (%s)", cudaGetErrorString(e));
    return DC_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lk(g_noalloc_mu);
  if (g_noalloc_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || p == nullptr) {
      dc::set_error("dc_conv_stack_noalloc: cudaGetSymbolAddress failed on device %d: %s", dev, cudaGetErrorString(e));
      return DC_ERR_CUDA;
    }
    g_noalloc_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return DC_OK;
}
}  // namespace

extern "C" dc_status dc_conv_stack_noalloc(const float* weights_dev, int hidden, int n_conv, const int* dilations,
                                           const float* x_dev, int n_frames, float* y_dev, void* cuda_stream) {
  if (!weights_dev || !dilations || !x_dev || !y_dev) {
    dc::set_error("dc_conv_stack_noalloc: null pointer argument");
    return DC_ERR_ARG;
  }
  if (hidden < 4 || hidden % 4 || n_conv < 1 || n_conv > DC_MAX_CONV || n_frames < 1) {
    dc::set_error("dc_conv_stack_noalloc: need hidden %% 4 == 0, 1 <= n_conv <= %d, n_frames >= 1", DC_MAX_CONV);
    return DC_ERR_ARG;
  }
  int dmax = 0;
  for (int l = 0; l < n_conv; ++l) {
    if (dilations[l] < 1 || dilations[l] > 4096) {
      dc::set_error("dc_conv_stack_noalloc: dilation %d out of range", dilations[l]);
      return DC_ERR_ARG;
    }
    dmax = dilations[l] > dmax ? dilations[l] : dmax;
  }
  const long long halo = 2ll * dmax;
  long long cap = 1;
  while (cap < (long long)n_frames + halo) cap <<= 1;
  const long long need = 2 * cap * hidden;
  if (need > (long long)DC_NOALLOC_SCRATCH_FLOATS) {
    dc::set_error("dc_conv_stack_noalloc: %d frames x %d channels with dilation %d need %lld scratch floats, "
                  "the built-in array holds %u", n_frames, hidden, dmax, need, DC_NOALLOC_SCRATCH_FLOATS);
    return DC_ERR_ARG;
  }
  float* scratch = nullptr;
  dc_status st = noalloc_scratch(&scratch);
  if (st != DC_OK) return st;
  cudaStream_t cs = (cudaStream_t)cuda_stream;
  float* region[2] = {scratch, scratch + cap * hidden};
  // The array keeps the previous call's values.  Rows [cap - halo, cap) of both regions are the
  // frames "before the start" that every block reads as its left context: they must be zero.
  for (int r = 0; r < 2; ++r) {
    cudaError_t e = cudaMemsetAsync(region[r] + (cap - halo) * hidden, 0, (size_t)(halo * hidden) * sizeof(float), cs);
    if (e != cudaSuccess) {
      dc::set_error("dc_conv_stack_noalloc: clearing the left context failed: %s", cudaGetErrorString(e));
      return DC_ERR_CUDA;
    }
  }
  size_t woff = 0;
  for (int l = 0; l < n_conv; ++l) {
    dc::TapConvF32 p{};
    // block l reads region[l & 1] (block 0: the caller's x, whose left context is the zeroed rows
    // of region[0]) and writes region[(l + 1) & 1] (last block: the caller's y)
    p.in_ring = region[l & 1];
    p.in_mask = (int)cap - 1;
    p.in_direct = (l == 0) ? x_dev : nullptr;
    p.pos_in = 0;
    p.T_in = n_frames;
    p.C_in = hidden;
    p.n_taps = 3;
    p.shift[0] = 2 * dilations[l]; p.shift[1] = dilations[l]; p.shift[2] = 0;
    p.n_phase = 1;
    p.W = weights_dev + woff;
    p.w_tap_stride = (long long)hidden * hidden;
    p.w_phase_stride = 0;
    woff += (size_t)3 * hidden * hidden;
    p.bias = weights_dev + woff;
    woff += (size_t)hidden;
    p.C_out = hidden;
    p.residual_silu = 1;
    if (l + 1 < n_conv) {
      p.out_ring = region[(l + 1) & 1];
      p.out_mask = (int)cap - 1;
    } else {
      p.out_direct = y_dev;
      p.pos_out = 0;
    }
    dc::launch_tapconv_f32(p, cs);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    dc::set_error("dc_conv_stack_noalloc: launch failed: %s", cudaGetErrorString(e));
    return DC_ERR_CUDA;
  }
  return DC_OK;
}
