// fp32 kernels of the conv pipeline and the vocoder tail: a tiled FFMA "tap GEMM" over ring
// buffers (causal conv k=3 with dilation, and the phases of the causal transposed conv), and the
// fused head conv + inverse STFT + overlap-add kernel.  fp32 parity (max err <= 1e-4 of RMS) rules
// out single-pass TF32, so these run on the FP32 pipe.
#include "dc_internal.h"
#include "dc_ptx.cuh"
#include "dc_rng.cuh"

#include <math.h>
#include <stdio.h>

#include <mutex>
#include <utility>

namespace dc {

namespace {

constexpr int BK = 32;   // reduction slice
constexpr int KQ = BK / 4;   // 16-byte copies per A-tile row

// SiLU through the special-function unit (ex2.approx and rcp.approx, each within 2 ulp): the libm forms cost about
// 25 instructions per element, a sixth of a small layer's instruction count; the error, a few 1e-7 relative, is far
// inside the 1e-4 budget of the fp32 configurations.
__device__ __forceinline__ float silu_f(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// Row of logical frame t: the caller's chunk for new frames of the first layer, else the ring.
__device__ __forceinline__ const float* in_row_ptr(const float* in_direct, long long pos_in, const float* in_ring, int in_mask,
                                                   int C_in, long long t) {
  if (in_direct != nullptr && t >= pos_in) return in_direct + (t - pos_in) * C_in;
  return in_ring + (long long)((int)(t & (long long)in_mask)) * C_in;
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros (out-of-range rows / columns).
__device__ __forceinline__ void cp_async16_zfill(void* dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
               "r"(src_bytes)
               : "memory");
}

// One CTA computes a BM x BN tile of one phase.  A group of BM*BN/16 threads (each a 4 x 4 micro
// tile) accumulates a share of the reduction; KS such groups split the reduction steps among
// themselves (step kb belongs to group kb % KS) and their partial tiles are summed through shared
// memory in a fixed order, so the result does not depend on timing.  The vocoder's early layers
// have few frames and long reductions: without the split most SMs would hold a single warp.
// Operands stream through a 3-stage cp.async ring per group (a reduction step is cheaper than one
// L2 round trip, so two steps are kept in flight).
constexpr int F32_STAGES = 3;

template <int BM, int BN>
struct TapTile {
  static constexpr int NTG = BM * BN / 16;                 // threads per group
  static constexpr int LDA = BK + 4;                       // row stride of the A tile (floats)
  static constexpr int STAGE_FLOATS = BM * LDA + BK * BN;  // one stage of one group
  static constexpr int GROUP_FLOATS = F32_STAGES * STAGE_FLOATS;
};

template <int BM, int BN>
__global__ void __launch_bounds__(512) tapconv_f32_kernel(const TapConvF32 p, const int KS) {
  using TT = TapTile<BM, BN>;
  ptx::pdl_launch();
  ptx::pdl_wait();          // the call record and the input ring come from earlier kernels
  // per-call values: by value, or from the device-side call record (captured graphs)
  int T_in = p.T_in;
  long long pos_in = p.pos_in, pos_out = p.pos_out;
  const float* in_direct = p.in_direct;
  float* out_direct = p.out_direct;
  int exc_rng_id = p.exc_rng_id;
  const float* in_ring = p.in_ring;
  float* out_ring = p.out_ring;
  float* save_ring = p.save_ring;
  int phase = blockIdx.z;
  const F32Call* callp = p.call;
  if (p.batch != nullptr) {
    const int slot = blockIdx.z / p.n_phase;
    phase = blockIdx.z - slot * p.n_phase;
    if (slot >= p.batch->n) return;
    const F32BatchSlot& bs = p.batch->s[slot];
    callp = &bs.call;
    in_ring = bs.ptrs->ring[p.layer];
    out_ring = p.last_layer ? nullptr : bs.ptrs->ring[p.layer + 1];
    save_ring = p.first_layer ? bs.ptrs->ring[p.layer] : nullptr;
  }
  if (callp != nullptr) {
    const F32Call c = *callp;
    exc_rng_id = c.rng_id;
    T_in = c.T * p.rate_in;
    pos_in = c.frames * p.rate_in;
    pos_out = pos_in * p.n_phase;
    in_direct = p.first_layer ? c.feats : nullptr;
    out_direct = p.last_layer ? c.out : nullptr;
  }
  if ((int)blockIdx.x * BM >= T_in) return;   // the grid is sized for the longest chunk
  const int in_mask = p.in_mask, C_in = p.C_in, C_out = p.C_out;
  const int sh0 = p.shift[0], sh1 = p.shift[1], sh2 = p.shift[2];
  constexpr int NTG = TT::NTG;
  constexpr int TX = BN / 4;              // threads along the channel axis
  constexpr int NA = BM * KQ / NTG;       // 16-byte copies of the A tile per thread
  constexpr int NB = BK * BN / 4 / NTG;   // 16-byte copies of the B tile per thread
  constexpr int LDA = TT::LDA;
  extern __shared__ __align__(16) float f32_smem[];

  const int grp = threadIdx.x / NTG;      // reduction group
  const int tid = threadIdx.x - grp * NTG;
  float* gbase = f32_smem + grp * TT::GROUP_FLOATS;
  const int tx = tid % TX, ty = tid / TX;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  const float* Wp = p.W + (long long)phase * p.w_phase_stride;

  const int kb_per_tap = (C_in + BK - 1) / BK;
  const int nkb = p.n_taps * kb_per_tap;
  const int my_steps = (nkb - grp + KS - 1) / KS;   // steps grp, grp + KS, ...

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  // Per-thread copy descriptors, hoisted out of the step loop: the source row of every A copy for
  // each tap, and the base of every B copy.
  const float* a_src[NA][3];
  bool a_ok[NA];
  int a_dst[NA], a_kq[NA];
#pragma unroll
  for (int u = 0; u < NA; ++u) {
    const int i = tid + u * NTG;
    const int row = i / KQ;
    a_kq[u] = (i % KQ) * 4;                               // A tile: BM rows x BK k
    a_ok[u] = m0 + row < T_in;
    a_dst[u] = row * LDA + a_kq[u];
    const long long t = pos_in + m0 + row;
    a_src[u][0] = in_row_ptr(in_direct, pos_in, in_ring, in_mask, C_in, t - sh0) + a_kq[u];
    a_src[u][1] = in_row_ptr(in_direct, pos_in, in_ring, in_mask, C_in, t - sh1) + a_kq[u];
    a_src[u][2] = in_row_ptr(in_direct, pos_in, in_ring, in_mask, C_in, t - sh2) + a_kq[u];
  }
  const float* b_src[NB];
  bool b_ok[NB];
  int b_dst[NB], b_k[NB];
#pragma unroll
  for (int u = 0; u < NB; ++u) {
    const int i = tid + u * NTG;
    b_k[u] = i / TX;                                      // B tile: BK k x BN n
    const int nq = (i % TX) * 4;
    b_ok[u] = n0 + nq < C_out;
    b_dst[u] = b_k[u] * BN + nq;
    b_src[u] = Wp + (long long)b_k[u] * C_out + n0 + nq;
  }
  const long long w_tap = p.w_tap_stride;

  auto issue = [&](int s) {   // s-th step of this group
    if (s < my_steps) {
      const int kb = grp + s * KS;
      float* As = gbase + (s % F32_STAGES) * TT::STAGE_FLOATS;   // [BM][LDA]
      float* Bs = As + BM * LDA;                                  // [BK][BN]
      const int tap = kb / kb_per_tap;
      const int c0 = (kb - tap * kb_per_tap) * BK;
#pragma unroll
      for (int u = 0; u < NA; ++u) {
        const bool ok = a_ok[u] && c0 + a_kq[u] < C_in;
        const float* src = (tap == 0 ? a_src[u][0] : (tap == 1 ? a_src[u][1] : a_src[u][2])) + c0;
        cp_async16_zfill(As + a_dst[u], ok ? src : p.W, ok ? 16 : 0);
      }
      const long long boff = (long long)tap * w_tap + (long long)c0 * C_out;
#pragma unroll
      for (int u = 0; u < NB; ++u) {
        const bool ok = b_ok[u] && c0 + b_k[u] < C_in;
        cp_async16_zfill(Bs + b_dst[u], ok ? b_src[u] + boff : p.W, ok ? 16 : 0);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");   // an (empty) group per step keeps the count uniform
  };

#pragma unroll
  for (int s = 0; s < F32_STAGES - 1; ++s) issue(s);
  for (int s = 0; s < my_steps; ++s) {
    asm volatile("cp.async.wait_group %0;" ::"n"(F32_STAGES - 2) : "memory");   // step s has landed
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(NTG) : "memory");       // for the whole group; step s-1's buffer is free
    issue(s + F32_STAGES - 1);
    const float* As = gbase + (s % F32_STAGES) * TT::STAGE_FLOATS;
    const float* Bs = As + BM * LDA;
#pragma unroll
    for (int k4 = 0; k4 < BK; k4 += 4) {
      float4 a[4];
#pragma unroll
      // (a thread's four rows are ty, ty + BM/4, ...: the four consecutive ty of a warp then read rows LDA = 36 words
      // apart, i.e. four different bank quads - with rows 4 ty + i two of them would share their banks)
      for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(As + (ty + (BM / 4) * i) * LDA + k4);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 b = *reinterpret_cast<const float4*>(Bs + (k4 + kk) * BN + tx * 4);
        const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float av = kk == 0 ? a[i].x : (kk == 1 ? a[i].y : (kk == 2 ? a[i].z : a[i].w));
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av, bv[j], acc[i][j]);
        }
      }
    }
  }

  if (KS > 1) {
    // fixed-order sum of the groups' partial tiles: group g parks its tile in its own (now idle)
    // operand ring, group 0 adds them in the order 1, 2, ...
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    if (grp > 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<float4*>(gbase + (tid * 4 + i) * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    }
    __syncthreads();
    if (grp > 0) return;
    for (int g = 1; g < KS; ++g) {
      const float* src = f32_smem + g * TT::GROUP_FLOATS;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float4 v = *reinterpret_cast<const float4*>(src + (tid * 4 + i) * 4);
        acc[i][0] += v.x; acc[i][1] += v.y; acc[i][2] += v.z; acc[i][3] += v.w;
      }
    }
  }

  const int n = n0 + tx * 4;
  if (n < C_out) {
    const float4 bias = *reinterpret_cast<const float4*>(p.bias + n);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = m0 + ty + (BM / 4) * i;
      if (row >= T_in) continue;
      const long long t_in = pos_in + row;
      float4 v = make_float4(acc[i][0] + bias.x, acc[i][1] + bias.y, acc[i][2] + bias.z, acc[i][3] + bias.w);
      if (p.residual_silu) {
        const float4 x = *reinterpret_cast<const float4*>(in_row_ptr(in_direct, pos_in, in_ring, in_mask, C_in, t_in) + n);
        v = make_float4(x.x + silu_f(v.x), x.y + silu_f(v.y), x.z + silu_f(v.z), x.w + silu_f(v.w));
      }
      if (p.post_silu) v = make_float4(silu_f(v.x), silu_f(v.y), silu_f(v.z), silu_f(v.w));
      const long long t_out = (long long)p.n_phase * t_in + phase;
      if (p.exc_std != 0.f) {   // the stream's clock at this layer's output rate is the generator's offset
        uint32_t w[4];
        float z[4];
        philox4x32_10((uint32_t)(unsigned long long)t_out, (uint32_t)((unsigned long long)t_out >> 32), (uint32_t)(n >> 2),
                      0x80000000u + (uint32_t)exc_rng_id, p.exc_seed_lo, p.exc_seed_hi, w);
        normals4(w, z);
        v.x = fmaf(p.exc_std, z[0], v.x); v.y = fmaf(p.exc_std, z[1], v.y); v.z = fmaf(p.exc_std, z[2], v.z); v.w = fmaf(p.exc_std, z[3], v.w);
      }
      float* dst = (out_direct != nullptr)
                       ? out_direct + (t_out - pos_out) * C_out + n
                       : out_ring + (long long)((int)(t_out & (long long)p.out_mask)) * C_out + n;
      *reinterpret_cast<float4*>(dst) = v;
    }
  }

  // Carry update of the first layer: its left context for the next chunk is the tail of the
  // caller's chunk, written into ring rows that no CTA of this launch reads (distinct logical
  // frames map to distinct rows because the ring holds f_chunk + halo frames).
  if (save_ring != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && phase == 0) {
    const int first = T_in > p.save_rows ? T_in - p.save_rows : 0;
    const int c4 = C_in >> 2;
    for (int i = tid; i < (T_in - first) * c4; i += NTG) {
      const int r = first + i / c4, c = (i - (i / c4) * c4) * 4;
      const float4 v = *reinterpret_cast<const float4*>(in_direct + (long long)r * C_in + c);
      *reinterpret_cast<float4*>(save_ring + (long long)((int)((pos_in + r) & (long long)in_mask)) * C_in + c) = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------

constexpr int HFR = 64;         // frames per CTA of the head kernel: 3 recomputed frames of overlap + 61 new ones
constexpr int HF = HFR - 3;     // new frames per CTA
constexpr int HQ = 4;           // threads per frame: each reduces a quarter of the channels, then a quarter of the DFT outputs
constexpr int HT = HFR * HQ;    // threads per CTA
constexpr int NFFT = 16, NB = 9, NH = 18, HOP = 4, TAIL = NFFT - HOP;

__constant__ float c_cos16[16];  // cos(2 pi j / 16)
__constant__ float c_sin16[16];
__constant__ float c_hann16[16];

// One thread per frame left a 3 x C x 18 reduction (3,456 dependent multiply-adds at C = 64) on two warps per CTA:
// 23 us for 6,000 frames.  Four adjacent lanes share a frame: lane q reduces the channels c = q (mod 4) blocks of
// four, the partial sums are added across the four lanes in a fixed butterfly (every lane ends with the same
// bits), and lane q then produces DFT outputs 4q .. 4q + 3 of the frame.
__global__ void __launch_bounds__(HT) head_istft_f32_kernel(const HeadIstftF32 p_in) {
  extern __shared__ __align__(16) float smem[];
  ptx::pdl_launch();
  ptx::pdl_wait();
  HeadIstftF32 p = p_in;
  if (p.batch != nullptr) {
    if ((int)blockIdx.y >= p.batch->n) return;
    const F32BatchSlot& bs = p.batch->s[blockIdx.y];
    p.call = &bs.call;
    p.in_ring = bs.ptrs->ring[p.layer];
    p.tails = bs.ptrs->tails;
  }
  if (p.call != nullptr) {
    const F32Call c = *p.call;
    p.T = c.T * p.rate_in;
    p.pos = c.frames * p.rate_in;
    p.tail_in = p.tails + 12 * c.parity;
    p.tail_out = p.tails + 12 * (c.parity ^ 1);
    p.pcm = c.out;
  }
  if ((int)blockIdx.x * HF >= p.T) return;
  float* Ws = smem;                              // [3*C][NH]
  float* g = smem + 3 * p.C * NH;                // [HFR][NFFT] windowed frame signals
  const int tid = threadIdx.x;
  for (int i = tid; i < 3 * p.C * NH; i += HT) Ws[i] = p.W[i];
  __syncthreads();

  const int fr = tid / HQ, q = tid % HQ;          // frame slot of the CTA, quarter
  const int f_local = blockIdx.x * HF + fr - 3;   // frame index within the chunk (may be < 0)
  const bool compute = f_local >= 0 && f_local < p.T;   // frames of earlier chunks come from the tail
  // (all four lanes of a frame take the same branch, and a warp holds whole frames: the shuffles below are
  // executed by complete groups)
  float z[NH];
#pragma unroll
  for (int o = 0; o < NH; ++o) z[o] = 0.f;
  if (compute) {
    const long long t = p.pos + f_local;
    for (int tap = 0; tap < 3; ++tap) {
      const float* x = p.in_ring + (long long)((int)((t - (2 - tap)) & (long long)p.in_mask)) * p.C;
      const float* w = Ws + tap * p.C * NH;
      for (int c = 4 * q; c < p.C; c += 4 * HQ) {
        const float4 xv = *reinterpret_cast<const float4*>(x + c);
        const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int o = 0; o < NH; ++o) z[o] = fmaf(xs[u], w[(c + u) * NH + o], z[o]);
      }
    }
  }
#pragma unroll
  for (int o = 0; o < NH; ++o) {
    z[o] += __shfl_xor_sync(0xffffffffu, z[o], 1);
    z[o] += __shfl_xor_sync(0xffffffffu, z[o], 2);
  }
  float gv[NFFT / HQ];
#pragma unroll
  for (int k = 0; k < NFFT / HQ; ++k) gv[k] = 0.f;
  if (compute) {
    float re[NB], im[NB];
#pragma unroll
    for (int f = 0; f < NB; ++f) {
      const float mag = expf(fminf(z[f] + p.bias[f], p.clamp));
      float sn, cs;
      sincosf(z[NB + f] + p.bias[NB + f], &sn, &cs);
      re[f] = mag * cs;
      im[f] = mag * sn;
    }
#pragma unroll
    for (int kk = 0; kk < NFFT / HQ; ++kk) {
      const int k = q * (NFFT / HQ) + kk;
      float a = re[0] + ((k & 1) ? -re[NB - 1] : re[NB - 1]);
#pragma unroll
      for (int f = 1; f < NB - 1; ++f) {
        const int j = (f * k) & 15;
        a += 2.0f * (re[f] * c_cos16[j] - im[f] * c_sin16[j]);
      }
      gv[kk] = c_hann16[k] * a * (1.0f / NFFT);
    }
  }
#pragma unroll
  for (int kk = 0; kk < NFFT / HQ; ++kk) g[fr * NFFT + q * (NFFT / HQ) + kk] = gv[kk];
  __syncthreads();

  // overlap-add: one thread per new frame
  const int fo = tid;                              // frame slot
  const int fo_local = blockIdx.x * HF + fo - 3;
  if (tid < HFR && fo >= 3 && fo_local < p.T) {
    const float inv_norm = 1.0f / 1.5f;   // sum of the four overlapping squared Hann windows
    float out[HOP];
#pragma unroll
    for (int j = 0; j < HOP; ++j) {
      // sample 4 f + j: contributions of frames f, f-1, f-2, f-3 at offsets j, 4+j, 8+j, 12+j;
      // the part that frames of earlier chunks contribute is the carried tail
      float a = (fo_local < 3 && 4 * fo_local + j < TAIL) ? p.tail_in[4 * fo_local + j] : 0.f;
#pragma unroll
      for (int i = 3; i >= 0; --i) a += g[(fo - i) * NFFT + 4 * i + j];
      out[j] = a * inv_norm;
    }
    *reinterpret_cast<float4*>(p.pcm + 4ll * fo_local) = make_float4(out[0], out[1], out[2], out[3]);
    if (fo_local == p.T - 1) {
      // tail for the next chunk: samples 4T + q, q in [0,12), from the last three frames
      for (int qq = 0; qq < TAIL; ++qq) {
        float a = 0.f;
        for (int i = 2; i >= 0; --i)
          if (4 * (i + 1) + qq < NFFT) a += g[(fo - i) * NFFT + 4 * (i + 1) + qq];
        p.tail_out[qq] = a;
      }
    }
  }
}

}  // namespace

namespace {
__global__ void set_f32_call_kernel(const F32Call v, F32Call* dst) {
  ptx::pdl_launch();
  if (threadIdx.x == 0) *dst = v;
}

__global__ void set_f32_batch_kernel(const __grid_constant__ F32Batch v, F32Batch* dst) {
  if (threadIdx.x == 0) {
    dst->n = v.n;
    dst->pad = 0;
  }
  if ((int)threadIdx.x < v.n) dst->s[threadIdx.x] = v.s[threadIdx.x];
}

template <typename... KArgs, typename... Args>
void launch_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <int BM, int BN>
void launch_tile(const TapConvF32& p, int KS, int T_grid, cudaStream_t st, bool pdl, int n_batch) {
  using TT = TapTile<BM, BN>;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {   // opt in to > 48 KB of dynamic shared memory, once per device
    const int want = 8 * TT::GROUP_FLOATS * 4;
    cudaFuncSetAttribute(tapconv_f32_kernel<BM, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, want > 227 * 1024 ? 227 * 1024 : want);
    attr_set[dev] = true;
  }
  dim3 grid((T_grid + BM - 1) / BM, (p.C_out + BN - 1) / BN, p.n_phase * (n_batch > 0 ? n_batch : 1));
  launch_ex(tapconv_f32_kernel<BM, BN>, grid, dim3(KS * TT::NTG), (size_t)KS * TT::GROUP_FLOATS * sizeof(float), st, pdl, p, KS);
}
}  // namespace

const void* set_f32_call_func() { return (const void*)set_f32_call_kernel; }

void launch_set_f32_call(const F32Call& v, F32Call* dst, cudaStream_t st) {
  set_f32_call_kernel<<<1, 32, 0, st>>>(v, dst);
}

void launch_set_f32_batch(const F32Batch& v, F32Batch* dst, cudaStream_t st) {
  set_f32_batch_kernel<<<1, F32_MAX_BATCH, 0, st>>>(v, dst);
}
const void* set_f32_batch_func() { return (const void*)set_f32_batch_kernel; }

void launch_tapconv_f32(const TapConvF32& p, cudaStream_t st, int T_grid, bool pdl, int n_batch) {
  if (T_grid < 0) T_grid = p.T_in;
  const int nkb = p.n_taps * ((p.C_in + BK - 1) / BK);
  const long long ctas64 = (long long)((T_grid + 63) / 64) * ((p.C_out + 63) / 64) * p.n_phase;
  if (ctas64 >= 296) {
    launch_tile<64, 64>(p, 1, T_grid, st, pdl, n_batch);
  } else {
    // few tiles: small tiles, and split the reduction inside the CTA until the GPU holds about
    // 1200 warps (8 per SM), keeping at least 4 steps per group; at most 8 groups (512 threads)
    const long long ctas32 = (long long)((T_grid + 31) / 32) * ((p.C_out + 31) / 32) * p.n_phase;
    int KS = 1;
    while (KS < 8 && ctas32 * 2 * KS < 1200 && nkb / (2 * KS) >= 4) KS *= 2;
    launch_tile<32, 32>(p, KS, T_grid, st, pdl, n_batch);
  }
}

// ---- FP32 multiply-add peak, measured -----------------------------------------------------------------------
// Sixteen independent fused multiply-add chains per thread, 1,024 threads per SM-filling CTA pair: nothing but the FP32
// pipe limits it.  The result is written so that the compiler keeps the arithmetic.
__global__ void __launch_bounds__(512) fp32_peak_kernel(float* out, int iters, float a, float b) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) x[i] = (float)(threadIdx.x + i);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = fmaf(x[i], a, b);
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += x[i];
  if (s == 123.456f) out[blockIdx.x * blockDim.x + threadIdx.x] = s;   // (practically never: the store only keeps the loop alive)
}

cudaError_t measure_fp32_peak(double* tflops) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  float* d = nullptr;
  const int ctas = sms * 4, iters = 1 << 14;
  if (e == cudaSuccess) e = cudaMalloc(&d, (size_t)ctas * 512 * sizeof(float));
  cudaEvent_t a = nullptr, b = nullptr;
  if (e == cudaSuccess) e = cudaEventCreate(&a);
  if (e == cudaSuccess) e = cudaEventCreate(&b);
  double best = 0.0;
  for (int rep = 0; rep < 5 && e == cudaSuccess; ++rep) {   // the first repetitions also warm the clocks up
    cudaEventRecord(a);
    fp32_peak_kernel<<<ctas, 512>>>(d, iters, 0.999f, 0.001f);
    cudaEventRecord(b);
    e = cudaEventSynchronize(b);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
    const double fl = 2.0 * 16.0 * iters * 512.0 * ctas;
    if (e == cudaSuccess && ms > 0.f && fl / (ms * 1e-3) / 1e12 > best) best = fl / (ms * 1e-3) / 1e12;
  }
  if (a) cudaEventDestroy(a);
  if (b) cudaEventDestroy(b);
  if (d) cudaFree(d);
  *tflops = best;
  return e;
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

void launch_head_istft_f32(const HeadIstftF32& p, cudaStream_t st, int T_grid, bool pdl, int n_batch) {
  if (T_grid < 0) T_grid = p.T;
  const size_t smem = (size_t)(3 * p.C * NH + HFR * NFFT) * sizeof(float);
  const int grid = (T_grid + HF - 1) / HF;
  launch_ex(head_istft_f32_kernel, dim3(grid, n_batch > 0 ? n_batch : 1), dim3(HT), smem, st, pdl, p);
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
  if (((reinterpret_cast<uintptr_t>(weights_dev) | reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(y_dev)) & 15u) != 0) {
    dc::set_error("dc_conv_stack_noalloc: weights_dev, x_dev and y_dev must be 16-byte aligned (the kernels use 16-byte accesses)");
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
