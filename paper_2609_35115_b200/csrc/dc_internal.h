// Internal declarations shared by the translation units of libdc (not installed).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "dc.h"

namespace dc {

// ---------------------------------------------------------------------------------------------
// fp32 tap convolution over ring buffers (conv pipeline and vocoder tail)
// ---------------------------------------------------------------------------------------------
// A layer reads frames by logical index t (frames since stream start at that layer's rate).
// Frame t lives in row (t & mask) of a power-of-two ring; frames t >= pos_in may instead come
// from a plain [T_in][C_in] array (`in_direct`, the caller's chunk).  Rings start zeroed, so
// t < 0 reads the causal zero padding.  Nothing is ever concatenated or moved: the left context
// of the next chunk is simply the rows already in the ring.
// Per-call values of the fp32 pipelines, kept in device memory so that a captured graph of the
// chunk step stays valid from call to call: a tiny kernel rewrites this record (its by-value
// argument is the only thing that changes in the graph) and every layer kernel derives its frame
// counts, ring positions and the caller's pointers from it.
struct F32Call {
  long long    frames;     // frames decoded by the stream before this call
  int          T;          // frames presented by this call
  int          parity;     // which overlap-add tail buffer holds the previous call's tail
  const float* feats;      // caller's chunk
  float*       out;        // caller's output
  int          rng_id;     // the stream's device random stream (vocoder excitation)
};

// Several streams of one fp32 model in ONE launch of every layer (multi-session serving): a record per slot in
// device memory, rewritten per call by a setter kernel (its by-value argument), and - because every stream has
// rings of its own - a per-stream table of ring addresses written once at dc_stream_open.  Slot i of the batch
// is grid plane i of every layer kernel; the arithmetic of a slot is exactly that of a single-stream call.
constexpr int F32_MAX_LAYERS = 24;
constexpr int F32_MAX_BATCH = 64;
struct F32StreamPtrs {
  float* ring[F32_MAX_LAYERS];   // input ring of each layer
  float* tails;                  // [2][12] overlap-add tails
};
struct F32BatchSlot {
  F32Call              call;
  const F32StreamPtrs* ptrs;
};
struct F32Batch {
  int          n, pad;
  F32BatchSlot s[F32_MAX_BATCH];
};

struct TapConvF32 {
  const F32Batch* batch;   // if set: slot = blockIdx.z / n_phase; per-call values and ring addresses come from batch->s[slot]
  int          layer;      // ... ring[layer] is this layer's input ring, ring[layer + 1] its output ring
  const F32Call* call;     // if set: T_in, pos_in, pos_out, in_direct, out_direct come from *call
  int          rate_in;    // ... scaled by this layer's frames per chunk frame
  int          first_layer, last_layer;
  const float* in_ring;
  int          in_mask;
  const float* in_direct;     // may be null
  long long    pos_in;        // logical index of the first new input frame
  int          T_in;          // new input frames in this call
  int          C_in;
  int          n_taps;        // 3 (conv) or 2 (transposed conv phases)
  int          shift[3];      // tap j reads frame t - shift[j]
  int          n_phase;       // output frame index = n_phase * t + phase
  const float* W;             // weights of (phase p, tap j) at W + p*w_phase_stride + j*w_tap_stride, [C_in][C_out]
  long long    w_tap_stride;
  long long    w_phase_stride;
  const float* bias;          // [C_out]
  int          C_out;
  int          residual_silu; // out = in[t] + SiLU(acc + bias)   (needs C_in == C_out, n_phase == 1)
  int          post_silu;     // out = SiLU(out)
  float*       out_ring;      // row (t_out & out_mask)
  int          out_mask;
  float*       out_direct;    // or plain [T_out][C_out] rows (t_out - pos_out)
  long long    pos_out;
  float*       save_ring;     // if set: copy the last save_rows rows of in_direct into the input ring
  int          save_rows;
  // Random excitation added to this layer's output (vocoder: the last transposed conv): exc_std * N(0,1), the draw of
  // (output frame t, channels 4g..4g+3) being Philox4x32-10 at counter (t lo, t hi, g, 2^31 + rng id) under the seed.
  float        exc_std;       // 0: none
  uint32_t     exc_seed_lo, exc_seed_hi;
  int          exc_rng_id;    // by value, or from *call
};

// T_grid: frames the grid is sized for (p.T_in, or the largest T_in when p.call is set).
// n_batch > 0: the launch carries that many slots (p.batch set); tile shape and reduction split are those of the
// single-stream launch of the same layer, so that a slot's result has the single-stream bytes.
void launch_tapconv_f32(const TapConvF32& p, cudaStream_t st, int T_grid = -1, bool pdl = false, int n_batch = 0);
void launch_set_f32_call(const F32Call& v, F32Call* dst, cudaStream_t st);
const void* set_f32_call_func();
void launch_set_f32_batch(const F32Batch& v, F32Batch* dst, cudaStream_t st);
const void* set_f32_batch_func();

// Head conv (k = 3, input already SiLU-activated) + magnitude/phase -> inverse real DFT (n_fft = 16)
// -> synthesis window -> overlap-add (hop 4) with the 12-sample tail carried across chunks.
struct HeadIstftF32 {
  const F32Batch* batch;      // if set: slot = blockIdx.y; per-call values, ring and tails come from batch->s[slot]
  int          layer;
  const F32Call* call;        // if set: pos, T, tails and pcm come from *call
  int          rate_in;
  float*       tails;         // [2][12] ping-pong pair (used with call)
  const float* in_ring;       // [cap][C]
  int          in_mask;
  long long    pos;           // logical index of the first new frame
  int          T;             // new frames (>= 3)
  int          C;
  const float* W;             // [3][C][18]
  const float* bias;          // [18]
  float        clamp;         // upper clamp of the log-magnitude
  const float* tail_in;       // [12] unnormalised partial sums of samples hop*pos .. +11
  float*       tail_out;      // [12] the same for the next chunk (a different buffer)
  float*       pcm;           // [4*T]
};

void launch_head_istft_f32(const HeadIstftF32& p, cudaStream_t st, int T_grid = -1, bool pdl = false, int n_batch = 0);

// Uploads the constant tables of the head kernel (DFT twiddles, periodic Hann window) to the
// current device.  Synchronous; called from dc_create, never from a decode call.
cudaError_t prepare_f32_constants();
// Measured FP32 fused multiply-add throughput of the current device (TFLOP/s; a few milliseconds of device time).
cudaError_t measure_fp32_peak(double* tflops);

// ---------------------------------------------------------------------------------------------
// bf16 flow decoder (dc_flow.cu)
// ---------------------------------------------------------------------------------------------
struct DevBuf {
  void*  p;
  size_t bytes;
};

struct FlowModel;    // packed bf16 weights, tensor maps, timestep-bias table, scratch for max_batch streams
struct FlowState;    // carries of one stream

void set_error(const char* fmt, ...);

// Every device allocation of the library goes through this pair (dc_api.cu).  Two test facilities hang off it, both
// host-side: an injected allocation failure (dc_test_fail_allocation: the n-th allocation made by the calling thread
// from now on reports cudaErrorMemoryAllocation without touching the device) and guard zones (while guard mode is on
// for the calling thread - dc_stream_open of a model created with DC_OPT_GUARD_ZONES - an allocation gets 256 bytes
// of a known pattern in front of and behind it, which dc_stream_check_guards reads back).
cudaError_t dev_alloc(void** p, size_t bytes);
void        dev_free(void* p);
template <typename T>
inline cudaError_t dev_alloc(T** p, size_t bytes) { return dev_alloc(reinterpret_cast<void**>(p), bytes); }

dc_status flow_model_create(const dc_config& cfg, const float* w, FlowModel** out);
void      flow_model_destroy(FlowModel* m);
dc_status flow_state_open(FlowModel* m, FlowState** out);
void      flow_state_buffers(const FlowState* s, DevBuf* out, int max_entries, int* n);
long long flow_state_frames(const FlowState* s);              // the stream's frame clock (committed frames)
void      flow_state_set_frames(FlowState* s, long long frames);
int       flow_state_rng_id(const FlowState* s);               // which device random stream the session draws from
void      flow_state_set_rng_id(FlowState* s, int id);
dc_status flow_state_reset(FlowModel* m, FlowState* s, cudaStream_t st);
void      flow_state_close(FlowState* s);
// Reads (and clears) the device-side error word that bounded waits set; synchronous.  0 = no timeout.
dc_status flow_selftest_bounded_wait(int max_polls);
int       flow_take_device_error(FlowModel* m);
const int* flow_error_word(const FlowModel* m);   // device address of that word
uint64_t  flow_graph_launches(const FlowModel* m);   // graph launches issued by decode calls so far
// One chunk for each of n streams.  Returns the number of kernel launches through *launches.
dc_status flow_decode(FlowModel* m, int n, FlowState* const* states, const float* const* feats_dev,
                      const int* n_frames, float* const* out_dev, cudaStream_t st, int* launches);
// All of the remaining input of n_streams streams at once, n_steps chunks per stream in flight (one per Euler
// step); same bytes as chunk-by-chunk decoding.  feats rows are in_dim floats wide; outs[i] receives n_frames[i]
// mel rows.  on_chunk (may be null) is called on the host with (hook_ctx, stream index, j) right after the pass that
// finishes chunk j of that stream has been enqueued.
dc_status flow_decode_wave(FlowModel* m, int n_streams, FlowState* const* states, const float* const* feats_dev, int in_dim,
                           const long long* n_frames, float* const* outs_dev, cudaStream_t st, int* launches,
                           void (*on_chunk)(void*, int, long long) = nullptr, void* hook_ctx = nullptr);

// Event-bracketed launches while profiling is on (see dc_profile_begin in dc.h).
struct Profiler {
  bool on = false;
  int  used = 0, cap = 0;
  cudaEvent_t* ev = nullptr;     // 2 per launch
  int*         cls = nullptr;
};
void flow_set_profiler(FlowModel* m, Profiler* prof);

// Brackets one launch with events when profiling is on.
struct ProfScope {
  Profiler*    p;
  cudaStream_t st;
  int          idx = -1;
  ProfScope(Profiler* prof, int cls, cudaStream_t s) : p(prof), st(s) {
    if (p && p->on && p->used < p->cap) {
      idx = p->used++;
      p->cls[idx] = cls;
      cudaEventRecord(p->ev[2 * idx], st);
    }
  }
  ~ProfScope() {
    if (idx >= 0) cudaEventRecord(p->ev[2 * idx + 1], st);
  }
};

}  // namespace dc
