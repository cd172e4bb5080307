/*
 * dc.h - C ABI of the streaming decoder step (one GPU, sm_100a).
 *
 * One call of dc_decode_chunk / dc_decode_batch runs the whole per-chunk decoder
 * step on the device: for the flow decoder the input projection, the causal
 * conv residual blocks and chunk-causal attention over [carried state | new
 * chunk], repeated for every Euler step, with the Euler update; for the
 * vocoder tail the transposed-conv upsampler, the magnitude/phase head and the
 * inverse STFT with overlap-add.  All state that crosses chunks (conv left
 * context, key/value carry, overlap-add tail) lives in device buffers that are
 * allocated once per stream, keep their address for the stream's lifetime and
 * are read and written in place (paper Section 3.2, "State Rule", Eq. 4: the
 * carry is written into existing storage and its pointer stays constant; the
 * retained extent is capped after inference, Section 3.1 "Two extents").
 *
 * Conventions
 *   - All matrices are row-major, one frame per row, channels contiguous.
 *   - "dev" pointers are device pointers valid on the model's device, "host"
 *     pointers are ordinary host pointers.  The library never takes ownership
 *     of a caller buffer.
 *   - Alignment: every device pointer to floats that a caller passes (feats_dev,
 *     out_dev, weights_dev, x_dev, y_dev, and each element of the host arrays of
 *     device pointers) must be 16-byte aligned - the kernels access them with
 *     16-byte loads and stores; a misaligned pointer is refused with DC_ERR_ARG
 *     before anything is launched.  Host buffers (the *_host calls) need only
 *     float alignment: a page-locked buffer is accessed directly by the kernels
 *     when it is 16-byte aligned and staged otherwise.
 *   - Every function returns a dc_status; nothing throws or aborts.  Argument
 *     and admission checks run before any state is touched (fail closed, paper
 *     Section 3.3 admission clauses; the admission predicate is
 *     1 <= n_frames <= f_chunk, Section 3.1).
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and is asynchronous unless
 *     stated otherwise.  A model owns one set of scratch buffers: all decode
 *     calls on streams of one model must be ordered on the device (use one
 *     CUDA stream, or synchronise between calls).
 *   - There is no CPU fallback: without a usable sm_100 device every call that
 *     needs the device fails with DC_ERR_CUDA.
 */
#ifndef DC_H_
#define DC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dc_model  dc_model;   /* immutable after creation: packed weights, constant tables */
typedef struct dc_stream dc_stream;  /* mutable: every carry of one audio stream                   */

typedef enum dc_status {
  DC_OK = 0,
  DC_ERR_ARG = 1,      /* null pointer, bad size, bad batch                                  */
  DC_ERR_CONFIG = 2,   /* configuration outside what the kernels support                     */
  DC_ERR_FRAMES = 3,   /* admission predicate violated: n_frames < 1 or n_frames > f_chunk   */
  DC_ERR_OOM = 4,      /* device or host allocation failed                                   */
  DC_ERR_CUDA = 5,     /* a CUDA call failed (see dc_last_error)                             */
  DC_ERR_TIMEOUT = 6,  /* a bounded device-side wait gave up; the stream is poisoned         */
  DC_ERR_STATE = 7     /* closed or poisoned stream, or streams of different models          */
} dc_status;

enum { DC_PIPE_CONV = 1, DC_PIPE_FLOW = 2, DC_PIPE_VOCODER = 3, DC_PIPE_TOKEN2WAV = 4 };
enum { DC_F32 = 0, DC_BF16 = 1 };   /* DC_BF16: bf16 storage and operands, fp32 accumulation */

/* dc_config.options: switches for tests and measurements.  None of the first four (nor DC_OPT_CTA_PAIRS) changes a result
 * byte; DC_OPT_ROUNDED_NORM selects the other of two admissible roundings.  (There is no configuration
 * by environment variable.) */
enum {
  DC_OPT_NO_GRAPH     = 1,        /* decode calls issue their kernels one by one instead of one captured graph  */
  DC_OPT_NO_PDL       = 2,        /* no programmatic dependent launch between the kernels of a step             */
  DC_OPT_NO_ZEROCOPY  = 4,        /* the *_host calls always stage, also for page-locked caller buffers         */
  DC_OPT_SERIAL_TAILS = 8,        /* token2wav dc_decode_batch: the vocoder tails stream by stream, not batched */
  /* Flow decoder: the RMS-normalised activations are written as a tensor of their own, rounded to bf16, and
   * the projections read it - the storage-point reading of "bf16 activations" taken literally - instead of
   * the default, which folds the norm into the projection as a scale of its fp32 accumulator rows and so
   * skips that one rounding (results of the two forms differ by a few 1e-3 of RMS; the folded form costs one
   * kernel and one activation round trip less per norm).  DC_PIPE_TOKEN2WAV always builds its flow decoder
   * this way: the vocoder tail amplifies the flow stage's deviation several times. */
  DC_OPT_ROUNDED_NORM = 16,
  /* Debug aid (the stand-in for a memory checker): every device buffer of a stream opened on this model is
   * allocated with 256 bytes of a known pattern in front of it and behind it; dc_stream_check_guards reads the
   * patterns back.  An index error in a kernel that writes just outside a carry is then reported instead of
   * silently corrupting a neighbour. */
  DC_OPT_GUARD_ZONES = 32,
  /* Flow decoder: full batches run the conv and QKV GEMMs of two adjacent row tiles as ONE 256-row product on
   * a pair of SMs (tcgen05 cta_group::2; each CTA stages half of the weight tile).  The results are the same
   * bytes either way.  Off by default: on this part the pair's fixed costs (cluster barrier before the odd
   * CTA's first copy, pair allocation of tensor memory) exceed what the shorter main loop saves for the
   * 7-microsecond kernels of this decoder. */
  DC_OPT_CTA_PAIRS = 64,
  /* MEASUREMENT ONLY - the outputs of such a model are meaningless: the step without the kernels of
   * one class, so that step-time differences give that class's cost inside the captured graph. */
  DC_OPT_SKIP_CONV_GEMM = 1 << 16,
  DC_OPT_SKIP_ATTENTION = 1 << 17,
  /* ... and the step whose GEMM and attention kernels return at once: same graph, same node count,
   * same launch attributes; its time divided by the node count is the cost of a bare stage boundary
   * (the t_sync of the stage-latency floor n_stages x t_sync; paper Section 2.2, T_o = sum t_k + G_o). */
  DC_OPT_EMPTY_KERNELS  = 1 << 18
};

#define DC_MAX_CONV 32
#define DC_MAX_UP 4
#define DC_MAX_RES 4

/* Plain-data description of the network.  Unused fields are zero.
 *   DC_PIPE_CONV    : hidden, n_conv, dilations[]           (fp32)
 *   DC_PIPE_FLOW    : hidden, n_conv, dilations[], n_attn, n_heads, head_dim, kv_cap,
 *                     n_steps, mel_dim                       (bf16)
 *   DC_PIPE_VOCODER : mel_dim, n_up, up_strides[], up_channels[n_up+1], n_res,
 *                     res_dilations[], n_fft, hop, logmag_clamp   (fp32)
 *   DC_PIPE_TOKEN2WAV : the fields of DC_PIPE_FLOW and of DC_PIPE_VOCODER (same mel_dim), precision
 *                     DC_BF16: the whole decoder step of the paper's segment (Section 2.2: flow
 *                     decoder, then vocoder and inverse STFT) in one call - a chunk of
 *                     [conditioning | noise] frames in, PCM out; the mel frames in between stay in a
 *                     device buffer of the stream (bf16 flow decoder, fp32 vocoder tail).  Weights:
 *                     the flow blob followed by the vocoder blob.  dc_decode_batch and dc_decode_batch_host
 *                     serve it too (max_batch <= 64).
 * The flow decoder runs n_conv / n_attn conv blocks, then one attention layer,
 * repeated n_attn times (n_attn = 0: conv blocks only). */
typedef struct dc_config {
  uint32_t size;                 /* sizeof(dc_config), for versioning                        */
  int32_t  pipeline;             /* DC_PIPE_*                                                */
  int32_t  precision;            /* DC_F32 | DC_BF16                                         */
  int32_t  hidden;               /* C                                                        */
  int32_t  n_conv;               /* causal conv residual blocks (k = 3)                      */
  int32_t  dilations[DC_MAX_CONV];
  int32_t  n_attn, n_heads, head_dim;
  int32_t  kv_cap;               /* W: carried key/value frames per (step, layer)            */
  int32_t  n_steps;              /* Euler steps per chunk                                    */
  int32_t  f_chunk;              /* largest admitted n_frames                                */
  int32_t  mel_dim;
  int32_t  n_up;
  int32_t  up_strides[DC_MAX_UP];
  int32_t  up_channels[DC_MAX_UP + 1];
  int32_t  n_res;
  int32_t  res_dilations[DC_MAX_RES];
  int32_t  n_fft, hop;
  float    rms_eps;
  float    logmag_clamp;
  int32_t  max_batch;            /* most streams one dc_decode_batch call may carry (>= 1)   */
  int32_t  f_prompt;             /* flow decoder: the stream's first f_prompt frames are a prompt whose keys/values
                                  * are never evicted; behind them the carry keeps the last kv_cap frames (the
                                  * paper's f_prompt + f_retained carry, Section 3.1 and Eq. 4).  0: a plain
                                  * sliding window of kv_cap frames.                              */
  int32_t  f_lookahead;          /* flow decoder: a call may present up to f_chunk + f_lookahead frames; the frames
                                  * beyond f_chunk are look-ahead (Section 3.1, "Two extents": they sit in the
                                  * envelope, the call attends them, and they are dropped before the retention
                                  * policy truncates): the call commits - output, conv left context, K/V carry -
                                  * its first min(n_frames, f_chunk) frames, reports that count through n_out, and
                                  * the caller presents the other frames again at the head of its next call.
                                  * f_chunk + f_lookahead <= 56.                                  */
  uint32_t noise_seed_lo, noise_seed_hi;   /* flow decoder: a non-zero 64-bit seed makes the decoder draw the Euler noise x_0
                                  * itself, so that a chunk's input is the conditioning alone ([n_frames][mel_dim]).
                                  * The draw for (frame t of the stream, channels 4g..4g+3) is Philox4x32-10 at counter
                                  * (t mod 2^32, t div 2^32, g, stream index) under the key (seed_lo, seed_hi): the
                                  * generator's offset is the stream's frame clock, so the captured chunk-step graph
                                  * draws exactly what direct launches would (the device-randomness clause of the
                                  * paper's effect classification, Section 3.3).  Four normals per draw by two
                                  * Box-Muller pairs on u = ((r >> 8) + 1/2) 2^-24.  The stream index is the number
                                  * of streams opened on the model before this one; snapshots carry it along.      */
  float    cfg_scale;            /* flow decoder: classifier-free guidance weight w >= 0; 0 = off.  With w > 0 every
                                  * Euler step evaluates the network twice - with the conditioning and with the
                                  * conditioning set to zero, each pass with carries of its own - and advances
                                  * x by ((1 + w) v_cond - w v_uncond) / n_steps (paper Table 1 measures the flow
                                  * step in this guided, batch x 2 form).  The two passes of a stream are two
                                  * row blocks of the same GEMM tiles.                            */
  int32_t  max_wave_frames;      /* token2wav pipeline: the most frames one dc_decode_wavefront call may carry per
                                  * stream.  dc_stream_open allocates the buffer that holds a wavefront call's mel
                                  * frames ([max_wave_frames][mel_dim] fp32) and the side stream its vocoder tails run
                                  * on, so that no decode call allocates; 0 = wavefront calls on this model are
                                  * refused.  Must be 0 for the other pipelines (their wavefront needs no buffer). */
  uint32_t options;              /* DC_OPT_* bits, 0 for normal use                           */
  float    excitation_std;       /* vocoder tail (and token2wav): > 0 adds a random excitation drawn on the device - the
                                  * vocoder's source signal, the paper's own instance of device randomness (Section
                                  * 3.1 "device random stream"; Section 3.3, effect classification: admitted because the
                                  * generator's offset is a function of the call clock).  The output of the LAST
                                  * transposed conv, before that stage's residual blocks, receives
                                  * excitation_std * N(0,1): the draw of (frame t at that layer's output rate, counted
                                  * from the stream start, channels 4g..4g+3) is Philox4x32-10 at counter
                                  * (t mod 2^32, t div 2^32, g, 2^31 + stream index) under the key below, four
                                  * normals per draw as for noise_seed.  Chunking, graph replay and snapshots cannot
                                  * change the draw.  0: no excitation (the five benchmark configurations).       */
  uint32_t excitation_seed_lo, excitation_seed_hi;   /* its key; non-zero when excitation_std > 0                */
} dc_config;

/* Number of floats of the canonical weight blob for this configuration, 0 if the
 * configuration is invalid.  Blob order (all matrices [C_in][C_out], conv and
 * transposed-conv weights tap-major [tap][C_in][C_out], tap 2 of a conv = current
 * frame):
 *   conv    : per block W[3][C][C], b[C]
 *   flow    : W_in[2 mel][C], b_in[C]; per group: per conv block W[3][C][C], b[C],
 *             P[C][C] (timestep bias tau = emb(t_s) P); then W_q, W_k, W_v, W_o [C][C],
 *             b_q, b_k, b_v, b_o [C]; finally W_out[C][mel], b_out[mel]
 *   vocoder : W_pre[3][mel][C0], b; per stage Wt[2 stride][C_in][C_out], b, per residual
 *             block W[3][C_out][C_out], b; W_head[3][C_last][n_fft+2], b. */
size_t dc_weights_count(const dc_config* cfg);

/* Builds a model on the current CUDA device: validates cfg, converts and packs
 * the weights (bf16 round-to-nearest-even for DC_BF16), precomputes the constant
 * tables (per-step timestep bias, synthesis window) and allocates the scratch
 * buffers for max_batch streams.  weights_host: n_floats floats in the canonical
 * order; the caller may free it on return.  Synchronous.  (Device-resident
 * constants: paper Section 3.1, "constant has a trivial clock".) */
dc_status dc_create(const float* weights_host, size_t n_floats, const dc_config* cfg, dc_model** out);

/* Frees a model: the shared binding of Section 3.4 (weights, constant tables, captured graphs) goes
 * when the last session has gone.  All its streams must be closed first (else DC_ERR_STATE). */
dc_status dc_destroy(dc_model* model);

/* Allocates and zeroes every carry of one stream (conv left context per (step,
 * block), key/value ring per (step, attention layer), vocoder left contexts,
 * overlap-add tail).  The buffers never move until dc_stream_close (paper
 * Section 3.2: pointer constancy over the stream lifetime).  Synchronous. */
dc_status dc_stream_open(dc_model* model, dc_stream** out);

/* Turn boundary: writes the base state (zeros, empty key/value carry) into the
 * existing buffers, on cuda_stream; addresses do not change (Section 3.2). */
dc_status dc_stream_reset(dc_stream* stream, void* cuda_stream);

/* Ends the stream and frees its carries (the per-session state of Section 3.4 ends with the session);
 * the handle stays recognisable as closed (DC_ERR_STATE) until dc_destroy. */
dc_status dc_stream_close(dc_stream* stream);

/* One chunk of one stream.
 *   feats_dev : device fp32 [n_frames][F_in]; F_in = hidden (conv), 2*mel_dim (flow and token2wav:
 *               cols [0,mel) conditioning, [mel,2 mel) initial noise; mel_dim - the conditioning
 *               alone - when the model draws the noise itself, see noise_seed), mel_dim (vocoder)
 *   out_dev   : device fp32; conv: [n_frames][hidden]; flow: [committed frames][mel_dim];
 *               vocoder and token2wav: committed frames * prod(up_strides) * hop PCM samples
 *   n_out     : host pointer (may be NULL) receiving the number of floats written
 * Fails with DC_ERR_FRAMES unless 1 <= n_frames <= f_chunk + f_lookahead; a failed call leaves
 * the stream untouched.  The call commits min(n_frames, f_chunk) frames (see f_lookahead; all of
 * them when f_lookahead = 0).  Allocates nothing. */
dc_status dc_decode_chunk(dc_stream* stream, const float* feats_dev, int n_frames,
                          float* out_dev, int* n_out, void* cuda_stream);

/* One chunk for each of n distinct streams of one model (n <= max_batch) in one
 * pass; stream i consumes n_frames[i] frames from feats_dev[i] and writes
 * out_dev[i].  feats_dev, n_frames and out_dev are HOST arrays (of device
 * pointers / ints).  Results are bitwise identical to n single dc_decode_chunk
 * calls.  (Multi-session serving over shared weights with per-session state:
 * paper Section 3.4, last paragraph, and Section 4.3 "Serving capacity".)  Every admitted call is ONE
 * CUDA graph launch: the chunk step is captured once per batch size - for 1 and max_batch streams at
 * dc_create, for any other n at the first call that carries n streams (that one call also pays the
 * capture; the graphs form the finite catalog of Section 3.3, Eq. 5) - and only the slot table
 * passed by value changes from call to call.  All four pipelines: the fp32 pipelines run every layer
 * once for the whole batch (a slot of the batch is a plane of the layer's grid, with the tiles and the
 * reduction split of the single-stream step; at most 64 streams), and the token2wav composite batches
 * the flow decoder and then the vocoder tails in the same way - a serving round of n sessions is two
 * graph launches. */
dc_status dc_decode_batch(dc_model* model, int n, dc_stream* const* streams,
                          const float* const* feats_dev, const int* n_frames,
                          float* const* out_dev, void* cuda_stream);

/* Offline decoding of one stream whose remaining input is all there: the n_frames frames are cut
 * into consecutive chunks of f_chunk frames (the last one shorter), each attending its f_lookahead
 * following frames where they exist, and decoded as a WAVEFRONT: chunk j runs Euler step s of the
 * flow decoder (Section 3.1's per-chunk loop) in pass j + s of the network, so that n_steps chunks
 * are in flight at once, one per step, as the slots of one launch.  Chunk j's step s needs only the
 * step-s carries that chunk j-1 left one pass earlier, so the result - and the stream's carries
 * afterwards - are bitwise those of the same chunks given to dc_decode_chunk one by one.
 *   feats_dev : device fp32 [n_frames][F_in] (as for dc_decode_chunk)
 *   out_dev   : device fp32; flow: [n_frames][mel_dim]; token2wav: n_frames * out_per_frame samples
 *   n_out     : host pointer (may be NULL) receiving the number of floats written
 * Flow and token2wav pipelines; the model must have been created with max_batch >= n_steps
 * (DC_ERR_ARG otherwise, stream untouched).  The token2wav composite keeps the call's mel frames
 * in a device buffer owned by the stream and sized at dc_stream_open from dc_config.max_wave_frames;
 * a call with more frames than that is refused with DC_ERR_ARG, the stream untouched.  Like every
 * decode call, this one allocates nothing.  The composite's vocoder tail has no
 * Euler loop to pipeline: chunk j's tail is enqueued, behind an event, on a CUDA stream owned by
 * the dc_stream as soon as the pass that finishes chunk j is, so it runs beside the flow decoder's
 * later passes; cuda_stream is made to wait for the last tail before the call returns, so work the
 * caller enqueues afterwards on cuda_stream sees the complete output. */
dc_status dc_decode_wavefront(dc_stream* stream, const float* feats_dev, long long n_frames,
                              float* out_dev, long long* n_out, void* cuda_stream);

/* dc_decode_wavefront for n distinct streams of one model at once: every pass of the network then
 * carries n_steps chunks of each stream (n * n_steps slots; needs max_batch >= n * n_steps and
 * n * n_steps * (2 with guidance) <= 64, DC_ERR_ARG otherwise with the streams untouched).
 * feats_dev, n_frames, out_dev are HOST arrays as for dc_decode_batch; streams may have different
 * lengths (a stream that has finished leaves holes in the later passes).  Results are bitwise those
 * of n dc_decode_wavefront calls, hence of chunk-by-chunk decoding.  The single-stream pass is
 * captured as a graph at dc_create; another stream count captures its pass at its first call. */
dc_status dc_decode_wavefront_batch(dc_model* model, int n, dc_stream* const* streams,
                                    const float* const* feats_dev, const long long* n_frames,
                                    float* const* out_dev, void* cuda_stream);

/* Convenience for callers with host buffers: copies feats_host to the device,
 * decodes, copies the result back and synchronises cuda_stream.  Uses staging
 * buffers owned by the stream (allocated at dc_stream_open).  Flow pipeline: a caller buffer that
 * is page-locked (cudaHostAlloc / cudaHostRegister, checked per call) is not staged at all - the
 * kernels read the chunk from it and write the mel rows into it across the bus.  Returns
 * DC_ERR_TIMEOUT (and poisons the stream until dc_stream_reset) if a bounded device-side wait
 * gave up. */
dc_status dc_decode_chunk_host(dc_stream* stream, const float* feats_host, int n_frames,
                               float* out_host, int* n_out, void* cuda_stream);

/* dc_decode_batch for callers with host buffers, all four pipelines: feats_host[i] / out_host[i] are host
 * pointers (pageable or pinned).  Flow pipeline: if every input (every output) buffer is page-locked, the
 * kernels read the chunks from (write the results into) the caller's buffers directly, with no
 * staging copy and no copy-engine transfer on that side.  Otherwise the call gathers the chunks
 * in a pinned buffer owned by the model, moves them to the device in one transfer, decodes the
 * batch, brings all results back in one transfer and scatters them.  Either way it synchronises
 * cuda_stream before it returns.  Returns DC_ERR_TIMEOUT (and poisons the
 * streams) if a bounded device-side wait gave up.  Calls on one model must not overlap. */
dc_status dc_decode_batch_host(dc_model* model, int n, dc_stream* const* streams,
                               const float* const* feats_host, const int* n_frames,
                               float* const* out_host, void* cuda_stream);

/* Per-kernel-class device timing, for roofline reports (the paper's
 * measurement model, Section 2.2, Eq. 1: stage time vs its roofline bound).  Between
 * dc_profile_begin and dc_profile_end every kernel launch of decode calls on this model is
 * bracketed by CUDA events on the launching stream (this slows the step down: never report
 * throughput from a profiled pass).  dc_profile_end synchronises the device and returns, per
 * class, the summed milliseconds and the launch count.  Classes: 0 conv GEMM, 1 other GEMMs
 * (input/QKV/output projections), 2 attention, 3 unused (the RMS norm is folded into the GEMMs),
 * 4 slot table + input prep,
 * 5 fp32 tap convolution, 6 fp32 head + inverse STFT, 7 conv / QKV GEMMs launched as CTA pairs
 * (DC_OPT_CTA_PAIRS; they then do not count in classes 0 and 1).
 * max_launches bounds the event pool allocated by dc_profile_begin. */
dc_status dc_profile_begin(dc_model* model, int max_launches);
dc_status dc_profile_end(dc_model* model, double ms[8], uint64_t launches[8]);

/* (The paper has no counterpart for this entry point; it exists for callers that cannot
 * allocate device memory.)
 *
 * Some callers of this library run where cudaMalloc is off limits: inside a region whose memory
 * budget is fixed up front, in a process that must not disturb another allocator's pool, or in a
 * real-time audio callback where an allocation's unbounded latency is unacceptable.  dc_create
 * and dc_stream_open allocate, so those callers cannot use the stream API.  For them this one call
 * runs the causal conv residual stack (the DC_PIPE_CONV network: n_conv blocks of
 * h <- h + SiLU(conv_k3,dilation(h) + b)) over ONE whole sequence with zero left context, and
 * keeps the activations that pass between blocks in a fixed array that is part of the library
 * image instead of in allocated buffers.  The call allocates nothing: no cudaMalloc, no cudaFree,
 * no allocating library routine.
 *
 *   weights_dev : DEVICE pointer, canonical conv blob (per block W[3][C][C], b[C]), fp32
 *   dilations   : HOST array of n_conv dilations (each >= 1)
 *   x_dev       : DEVICE fp32 [n_frames][hidden] input;  y_dev: DEVICE fp32 [n_frames][hidden] output
 *
 * Limit: the scratch array holds DC_NOALLOC_SCRATCH_FLOATS floats (2 MiB; every GPU that loads
 * the library carries it until the process exits).  A call needs 2 * P * hidden floats, where P
 * is the smallest power of two >= n_frames + 2 * max(dilations); larger requests are refused
 * with DC_ERR_ARG and a message (dc_last_error) that states the need and the limit.  hidden must
 * be a multiple of 4.
 *
 * The first call on a device looks up the array's device address (a synchronous runtime query,
 * made with that device current); make that first call outside any stream capture.  All calls on
 * a device share the one array, which still holds the previous call's values: the call itself
 * clears the rows that must read as zero, and two calls that overlap on the GPU (issued on
 * different CUDA streams without ordering) race on it - order them.  Work is enqueued on
 * cuda_stream; the result is ready when that stream reaches the end of the call's work. */
#define DC_NOALLOC_SCRATCH_FLOATS (1u << 19)
dc_status dc_conv_stack_noalloc(const float* weights_dev, int hidden, int n_conv, const int* dilations,
                                const float* x_dev, int n_frames, float* y_dev, void* cuda_stream);

/* Snapshot of a stream's state - every carry buffer and the stream's clocks - in device memory that
 * the library allocates (the per-session state of paper Section 3.4: sessions share the weights and
 * the captured graphs, a session is its snapshot).  dc_stream_restore writes a snapshot back IN
 * PLACE into the carries of `stream` (their addresses do not change), which may be the stream the
 * snapshot came from - rewinding it - or any other open stream of the same model - moving the
 * session.  Both enqueue device-to-device copies on cuda_stream; a snapshot may be restored any
 * number of times and must be released with dc_snapshot_free (before dc_destroy).  Errors:
 * DC_ERR_STATE for a closed stream or a snapshot of another model, DC_ERR_OOM. */
typedef struct dc_snapshot dc_snapshot;
dc_status dc_stream_snapshot(dc_stream* stream, dc_snapshot** out, void* cuda_stream);
dc_status dc_stream_restore(dc_stream* stream, const dc_snapshot* snapshot, void* cuda_stream);
dc_status dc_snapshot_free(dc_snapshot* snapshot);

/* Device addresses and byte sizes of the stream's carry buffers, for checks of the pointer
 * constancy that Section 3.2 (Eq. 4) demands over the stream's lifetime: writes up to max_entries (address, bytes) pairs into out and
 * the number of buffers into n_entries. */
dc_status dc_stream_carry_info(const dc_stream* stream, uint64_t* out, int max_entries, int* n_entries);

/* counters[0] chunks decoded, [1] frames decoded, [2] calls rejected (DC_ERR_FRAMES),
 * [3] calls rejected (other argument/state errors), [4] device timeouts (this call reads the
 * device-side error word synchronously, so it also reports timeouts of asynchronous decode calls),
 * [5] kernel launches issued (kernel nodes of graph launches included), [6] streams open,
 * [7] CUDA graph launches issued by decode calls (one per chunk step - the paper's one launch
 * per chunk, Section 3.3 "Granularity", Eq. 6; rejected calls by reason: Section 3.3's counted
 * refusal reasons). */
dc_status dc_get_counters(const dc_model* model, uint64_t counters[8]);

/* Measures the FP32 fused multiply-add throughput of the current device (TFLOP/s) with a register-only kernel of
 * independent FMA chains: the denominator of the fp32 pipelines' roofline fractions (the paper's measurement model,
 * Section 2.2, Eq. 1, needs a peak P for the pipe a stage runs on; for the FP32 pipe no measured figure is supplied,
 * so the library measures it).  Synchronous, a few milliseconds; allocates and frees a small device buffer. */
dc_status dc_measure_fp32_peak(double* tflops);

/* Checks the guard zones around every device buffer of the stream (carries, rings, tails, staging; a model created
 * with DC_OPT_GUARD_ZONES - otherwise there is nothing to check and the call returns DC_OK).  Synchronises the
 * device.  DC_OK if every pattern is intact, DC_ERR_STATE if not (*n_damaged, which may be NULL, receives the number of
 * overwritten zones).  (Fail-closed discipline, paper Section 3.3, applied to the library's own memory.) */
dc_status dc_stream_check_guards(dc_stream* stream, int* n_damaged);

/* Host-side fault injection for tests (the paper has no counterpart): the nth device allocation that the calling
 * thread makes through this library from now on fails as if the device were out of memory, without touching the
 * device (nth = 1: the next one; 0 disarms).  dc_create and dc_stream_open must then return DC_ERR_OOM with
 * everything they had allocated released. */
dc_status dc_test_fail_allocation(int nth);

/* Self-test of the bounded device-side wait that every pipeline barrier in the kernels uses (the
 * fail-closed discipline of paper Section 3.3, applied to the device): launches a one-CTA kernel
 * that waits, for at most max_polls polls (1 .. 1,000,000), on a barrier that nothing ever
 * completes.  The wait must give up by itself and report it: returns DC_ERR_TIMEOUT when it did
 * (the expected outcome), DC_OK if the wait claimed success, DC_ERR_CUDA on a launch problem.
 * Synchronous; the context stays usable afterwards. */
dc_status dc_selftest_bounded_wait(int max_polls);

const char* dc_status_str(dc_status s);

/* Text of the last CUDA or validation error on the calling thread ("" if none). */
const char* dc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif  /* DC_H_ */
