// bf16 flow decoder: host engine + kernels.
//
// Data layout.  Up to max_batch streams are served by one pass.  Every activation matrix is a
// bf16 row-major [GUARD + 64*slots][C] array: stream slot i owns the 64-row block starting at
// row GUARD + 64 i, whose rows 0..7 hold the conv left context (the last 8 block-input frames of
// the previous chunk, copied in from the stream's carry by the producing epilogue) and rows
// 8..8+T-1 the T <= 56 frames of the chunk.  A tap of a dilated conv is then a plain row shift
// of the whole matrix.  One CTA computes a 128 x BN output tile (two slots).
//
// GEMM kernel (640 threads, one CTA per SM): warp 0 = TMA producer of the A tiles, warp 2 = TMA
// producer of the weight tiles, warps 1 and 3 = UMMA issuers (even / odd reduction blocks into
// accumulators of their own in tensor memory), warps 4..19 = epilogue (one TMEM lane = one output
// row per thread, one 16-column chunk in four).  The three taps of a conv block are the column
// blocks of ONE 128 x 3BN x 16 UMMA per reduction step; the epilogue shifts the tap products by
// rows through shared memory and adds them.  The epilogues fuse bias, timestep bias, SiLU,
// residual, the carry update of the next conv block, the row statistics of the RMS norm, the
// in-place append of K/V rows to the stream's ring, and the Euler update.
#include <cuda.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <new>
#include <utility>
#include <vector>

#include "dc_internal.h"
#include "dc_ptx.cuh"
#include "dc_rng.cuh"

namespace dc {

namespace {

typedef __nv_bfloat16 bf16;

constexpr int GUARD = 8;        // zero rows in front of every activation matrix (tap shifts never go negative)
constexpr int SLOT_ROWS = 64;   // rows per stream slot: 8 left-context rows + up to 56 chunk rows
constexpr int HALO = 8;         // carried frames per (step, conv block); dilation <= 4 reads at most 8 back
constexpr int TILE_M = 128;
constexpr int KBLK = 64;        // bf16 elements per 128-byte swizzled smem row
constexpr int MAX_STAGES = 8;
constexpr int GEMM_TILE_SMEM = 88 * 1024;    // operand stages of the single-issuer GEMMs (a short reduction needs no deeper ring)
constexpr int A_ROWS = TILE_M;         // rows of an A box = rows of the output tile (the conv taps are shifted in the epilogue)
constexpr int A_BYTES = A_ROWS * 128;
constexpr int MAX_BN = 192;
constexpr int EPI_GROUPS = 4;           // epilogue warps per TMEM lane quarter: group g owns the 16-column chunks g, g + 4, ...
constexpr int EPI_THREADS = 128 * EPI_GROUPS;
constexpr int GEMM_THREADS = 128 + EPI_THREADS;   // warp 0 TMA (A), warps 1 and 3 UMMA issuers, warp 2 TMA (B), the rest epilogue
constexpr int MAX_SLOTS_PER_SET = 64;

enum GemmMode { MODE_INPROJ = 0, MODE_CONV = 1, MODE_QKV = 2, MODE_OPROJ = 3, MODE_OUT = 4 };

struct SlotInfo {
  int          T;         // frames presented by this stream in this call
  int          kv_head;   // ring row that receives the chunk's first history (non-prompt) K/V row
  int          kv_len;    // carried history rows attended (<= kv_cap), before this chunk
  int          pass;      // 0: conditional pass (or the only one); 1: the unconditional pass of a guided stream (mu = 0, no output)
  const float* feats;     // [T][2 mel]
  float*       out;       // [T][mel]
  bf16*        halo;      // stream carry: [n_steps][n_conv][8][C]
  bf16*        kv;        // stream carry: [n_steps][n_attn][2][P + Rk][C] (P prompt rows, then the history ring)
  int          n_prompt0; // prompt rows present before this chunk (<= P); the chunk's first P - n_prompt0 frames join them
  int          Tc;        // committed frames (<= T): the others are look-ahead - computed and attended, but neither output
                          // nor carried (their K/V rows are written past the ring head and overwritten by the next call)
  long long    frame0;    // index of the chunk's first frame in the stream (the frame clock)
  int          rng_id;    // the stream's device random stream
  // Wavefront decoding (several chunks of one stream in flight, each at an Euler step of its own): the slot's step
  // is folded into its halo / kv pointers by the host; what remains per slot is the timestep-bias row and two flags.
  int          tau_off;   // float offset of the slot's Euler step inside the timestep-bias table (0 when the launch's own step applies)
  int          flags;     // SLOT_FIRST: the prep kernel loads x_0 and mu; SLOT_LAST: the output projection also writes `out`
  int          pad;
};
constexpr int SLOT_FIRST = 1, SLOT_LAST = 2;

struct SlotSet {
  int      first, count;
  SlotInfo s[MAX_SLOTS_PER_SET];
};

struct GemmParams {
  int          mode;
  int          BN;              // output columns per CTA (multiple of 16, <= 128)
  int          n_issuers;       // 1 or 2 UMMA-issuing threads (2: even / odd reduction blocks, own accumulators)
  int          n_stages;        // TMA pipeline depth (<= MAX_STAGES, n_stages * stage bytes <= GEMM_TILE_SMEM)
  int          n_slots;
  int          n_kblocks;       // 64-wide channel blocks of the A matrix (one pipeline stage each)
  int          taps;            // 1, or 3 for the conv blocks (weights: K index = tap * 64 * n_kblocks + channel)
  int          shift[3];        // row shift of tap j (0..8)
  const float* bias;            // [N]
  const float* tau;             // [N] or null
  const bf16*  resid;           // residual source matrix (same row layout) or null
  bf16*        out;             // output activation matrix or null
  int          ld;              // row stride (elements) of resid / out / q
  const SlotInfo* slots;
  long long    halo_off;        // element offset of the next conv's carry inside SlotInfo::halo, or -1
  bf16*        q_out;           // MODE_QKV
  long long    kv_off;          // element offset of this (step, layer)'s K ring inside SlotInfo::kv
  int          kv_rs, kv_hs;    // K/V planes: elements between a head's consecutive rows / between heads
  int          dh_shift;        // log2(head_dim)
  int          Rk;              // ring rows
  int          P;               // prompt rows in front of the ring (0: none)
  int          C;
  float*       xstate;          // MODE_OUT: fp32 Euler state [rows][mel]
  bf16*        ain;             // MODE_OUT: next step's input-projection operand [GUARD+rows][ld_ain]
  int          ld_ain;
  float        inv_n;
  int          last_step;
  int          mel;
  float        cfg_w;           // MODE_OUT: guidance weight; > 0: the tile's slots are the (conditional, unconditional) passes of one stream
  // RMS normalisation, folded into the GEMMs around it (Sec. 3.2 block form; the norm has no gain):
  // (x / rms(x)) W = (x W) / rms(x), so the GEMM that consumes a normalised operand reads x itself
  // and scales its accumulator rows, and the GEMM that produced x leaves the row sums of squares.
  // Partial sums are kept per 16-column chunk, [C / 16][ssq_ld], and added in chunk order, so the
  // statistic does not depend on the tile width chosen for the batch size.
  float*       ssq_out;         // producer: partial sums of squares of the stored (bf16) output, or null
  const float* ssq_in;          // consumer (MODE_QKV, MODE_OUT): partial sums of the operand rows
  long long    ssq_ld;          // rows per chunk plane
  float        inv_C, eps;
  int*         err;
  int          empty;           // measurement only: the kernel returns at once (the cost of the bare stage boundary)
};

// SiLU(z) = z * sigmoid(z) = 0.5 z (1 + tanh(z / 2)): one MUFU op per element instead of two (exp + reciprocal);
// the epilogue of a 128 x 64 tile is bound by the special-function unit.  tanh.approx has a relative
// error of about 2^-11, below the bf16 rounding of the stored result.
__device__ __forceinline__ float silu_f(float z) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * z));
  const float h = 0.5f * z;
  return fmaf(h, t, h);
}

__device__ __forceinline__ void pack16_bf16(const float* v, uint4& a, uint4& b) {
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  a = make_uint4(w[0], w[1], w[2], w[3]);
  b = make_uint4(w[4], w[5], w[6], w[7]);
}
__device__ __forceinline__ void store16(bf16* p, const uint4& a, const uint4& b) {
  *reinterpret_cast<uint4*>(p) = a;
  *reinterpret_cast<uint4*>(p + 8) = b;
}

// PAIR: the CTAs of two adjacent row tiles (a cluster of two along x, one TPC) run ONE 256-row UMMA per
// reduction step.  Each stages its own activation rows and only HALF of the weight tile (tmB then has boxes
// of BN / 2 rows), so a CTA draws 28 KB instead of 40 KB per reduction block from L2 and the whole weight
// panel of a C = 512 layer fits its shared memory ahead of the activations.  The even CTA issues for both;
// accumulators, epilogue and summation order are those of the single-CTA form, so the results are the same bits.
// Measured on the 32-stream serving workload: the main loop of a conv block drops from 3.9 k to 3.3 k cycles
// (400 per reduction block, the tensor pipe's own rate), but the odd CTA may not copy before the cluster barrier
// has told it that the even CTA's barriers exist, and that barrier, with the pair allocation of tensor memory,
// puts the first full stage 0.4 to 1.6 microseconds later - more than the loop saves in a 7-microsecond kernel.
// Hence an option (DC_OPT_CTA_PAIRS), off by default.
template <bool PAIR, int MODE_T, int BN_T = 0>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
flow_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // MODE_T >= 0: a kernel specialised for one role, so that the other roles' epilogues and the slot fields only they
  // use cost neither registers nor instructions
  const int mode = MODE_T >= 0 ? MODE_T : p.mode;
  const int n_taps = MODE_T == MODE_CONV ? 3 : (MODE_T >= 0 ? 1 : p.taps);
  const int n_iss = MODE_T == MODE_CONV ? 2 : p.n_issuers;
  const int BN = BN_T > 0 ? BN_T : p.BN;   // BN_T > 0: the tile width known at compile time (the chunk loop of the epilogue unrolls away)
  if (p.empty) {
    ptx::pdl_launch();
    ptx::pdl_wait();
    return;
  }
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // stage = [A tile 128 x 128 B | one B tile BN x 128 B per tap]; all tile sizes are multiples of
  // 1024 B.  The weight tiles of a conv block's three taps are adjacent, so that they form one
  // operand of 3 BN rows.
  // (PAIR: a "tile" is one of the CTA's `taps` units of BN / 2 weight rows; BN is then a multiple of 16)
  const uint32_t b_bytes = PAIR ? (uint32_t)BN * 64u : (uint32_t)BN * 128u;
  const uint32_t b_tile = (b_bytes + 1023u) & ~1023u;
  const uint32_t stage_bytes = (uint32_t)A_BYTES + (uint32_t)n_taps * b_tile;
  const int STAGES = p.n_stages;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * stage_bytes);
  uint64_t* empty = full + MAX_STAGES;
  uint64_t* accum = empty + MAX_STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  int* s_fail = reinterpret_cast<int*>(tmem_slot + 1);
  float* s_bias = reinterpret_cast<float*>(s_fail + 1);
  float* s_tau = s_bias + MAX_BN;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * TILE_M, n0 = blockIdx.y * BN;
  const uint32_t pair_rank = PAIR ? ptx::cluster_ctarank() : 0u;   // 0: issues the UMMAs and owns the "full" barriers
  // Accumulator: BN columns, or 3 BN for a conv block, whose three taps are the column blocks of ONE
  // product Z = X [W_0 | W_1 | W_2] (a row shift commutes with the product, so the taps are shifted
  // and added in the epilogue; a tcgen05.mma costs about 47 cycles however small it is, and one
  // 128 x 3BN x 16 instruction replaces three 128 x BN x 16 ones).  The second issuer's accumulator
  // sits acc2_off columns after the first.
  const uint32_t acc_w = (uint32_t)(n_taps * BN);
  const uint32_t acc2_off = acc_w <= 32 ? 32u : (acc_w <= 64 ? 64u : (acc_w <= 128 ? 128u : 256u));
  const uint32_t need_cols = n_iss == 2 ? 2u * acc2_off : acc_w;
  const uint32_t tmem_cols = need_cols <= 32 ? 32u : (need_cols <= 64 ? 64u : (need_cols <= 128 ? 128u : (need_cols <= 256 ? 256u : 512u)));

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      ptx::mbar_init(&full[i], 2);   // one arrival per producer thread
      ptx::mbar_init(&empty[i], 1);
    }
    ptx::mbar_init(accum, (uint32_t)n_iss);
    *s_fail = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    if (PAIR) ptx::tmem_alloc_pair(tmem_slot, tmem_cols);
    else ptx::tmem_alloc(tmem_slot, tmem_cols);
  }
  // PAIR: the CTAs signal each other's barriers and the even one writes both accumulators, so each must know
  // that the other's barriers and tensor memory exist.  Every thread arrives at the cluster barrier here
  // (thread 0 after the initialisation, warp 1 after the allocation) and waits only where it first depends
  // on the partner, which keeps most of the barrier's latency off the path to the first copy.
  if (PAIR) ptx::cluster_arrive();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch();   // the next kernel may start its prologue and its weight prefetch now

  if (warp == 0 || warp == 2) {
    // two producer threads, one per tensor map: warp 0 streams the A tiles, warp 2 the weight tiles.
    // The loops keep their state in registers (no division, no parameter reloads): a single thread
    // issues every copy, so its instruction count is what bounds the fill rate.
    {
      const uint32_t on = lane == 0;   // the whole warp runs the loop, lane 0 issues
      const bool is_a = warp == 0;
      const int nkb = p.n_kblocks, taps = n_taps;
      const int ya = GUARD + m0;
      // PAIR: the even CTA's barrier counts the bytes of both CTAs' copies; the odd CTA only issues its own
      const uint32_t tx_bytes = (is_a ? (uint32_t)A_BYTES : (uint32_t)taps * b_bytes) * (PAIR ? 2u : 1u);
      uint8_t* dst = smem + (is_a ? 0 : A_BYTES);
      // PAIR: this CTA's j-th weight unit is unit u = taps * rank + j of the 2 * taps half-tiles: tap u / 2, half u % 2
      int ux[3] = {0, 0, 0}, uy[3] = {0, 0, 0};
      if (PAIR) {
#pragma unroll
        for (int j = 0; j < 3; ++j) {
          const int u = taps * (int)pair_rank + j;
          ux[j] = (u >> 1) * nkb * KBLK;
          uy[j] = n0 + (u & 1) * (BN >> 1);
        }
      }
      const uint32_t full0 = PAIR ? ptx::map_to_cta(ptx::smem_u32(&full[0]), 0u) : 0u;
      int st = 0;
      uint32_t phase = 1;          // parity of the "empty" phase to wait for (first pass: no wait)
      int x = 0;
      if (PAIR && pair_rank != 0) ptx::cluster_wait();   // this CTA's copies count on its partner's barriers
      if (is_a) ptx::pdl_wait();   // activations come from the previous kernel; weights do not
      for (int kb = 0; kb < nkb; ++kb) {
        if (kb >= STAGES && !ptx::mbar_wait(&empty[st], phase)) {
          atomicCAS(p.err, 0, 1 | (is_a ? 0 : 0x10) | (mode << 8) | (kb << 12) | ((int)blockIdx.x << 20));
          *s_fail = 1;
          break;
        }
        if (PAIR) {
          ptx::mbar_expect_tx_if(on && pair_rank == 0, &full[st], tx_bytes);
          const uint32_t bar = full0 + (uint32_t)st * 8u;
          if (is_a) {
            ptx::tma_load_2d_pair_if(on, dst, &tmA, x, ya, bar);
          } else {
            ptx::tma_load_2d_pair_if(on, dst, &tmB, x + ux[0], uy[0], bar);
            if (taps == 3) {
              ptx::tma_load_2d_pair_if(on, dst + b_tile, &tmB, x + ux[1], uy[1], bar);
              ptx::tma_load_2d_pair_if(on, dst + 2 * b_tile, &tmB, x + ux[2], uy[2], bar);
            }
          }
        } else if (is_a) {
          ptx::mbar_expect_tx_if(on, &full[st], tx_bytes);
          ptx::tma_load_2d_if(on, dst, &tmA, x, ya, &full[st]);
        } else {
          ptx::mbar_expect_tx_if(on, &full[st], tx_bytes);
          ptx::tma_load_2d_if(on, dst, &tmB, x, n0, &full[st]);
          if (taps == 3) {
            ptx::tma_load_2d_if(on, dst + b_tile, &tmB, x + nkb * KBLK, n0, &full[st]);
            ptx::tma_load_2d_if(on, dst + 2 * b_tile, &tmB, x + 2 * nkb * KBLK, n0, &full[st]);
          }
        }
        x += KBLK;
        dst += stage_bytes;
        if (++st == STAGES) {
          st = 0;
          dst -= (size_t)STAGES * stage_bytes;
          phase ^= 1;
        }
      }
    }
  } else if (warp == 1 || warp == 3) {
    // UMMA issuers.  A single thread spends about 100 cycles per tcgen05.mma it issues, more than a
    // narrow UMMA takes to execute, so two warps issue alternate reduction blocks into accumulators
    // of their own; the epilogue adds the two in a fixed order.
    const int me = warp >> 1;                     // 0 or 1
    if (me < n_iss && pair_rank == 0) {
      const uint32_t on = lane == 0;
      // the weight tiles of the taps are adjacent in the stage (BN rows of 128 B each, BN a multiple of 8),
      // so together they are one K-major operand of taps * BN rows
      const uint32_t idesc = ptx::umma_idesc_bf16(PAIR ? 2 * TILE_M : TILE_M, n_taps * BN, 0, 0);
      // PAIR: every completion is reported to both CTAs (their producers and epilogues wait on barriers of their own)
      const uint32_t empty_mine = ptx::smem_u32(&empty[0]), empty_peer = PAIR ? ptx::map_to_cta(empty_mine, 1u) : 0u;
      const int nkb = p.n_kblocks, step = n_iss;
      const uint32_t d_acc = tmem_base + (uint32_t)me * acc2_off;
      // descriptor start addresses are in 16-byte units: +2 per 32-byte K step
      const uint64_t d_a0 = ptx::umma_desc_sw128(ptx::smem_u32(smem));
      const uint32_t stage16 = stage_bytes >> 4, ab16 = A_BYTES >> 4;
      uint32_t acc = 0;
      if (PAIR) ptx::cluster_wait();   // the partner's tensor memory and barriers
      for (int kb = me; kb < nkb; kb += step) {
        const int st = kb % STAGES;
        if (!ptx::mbar_wait(&full[st], (uint32_t)(kb / STAGES) & 1u)) {
          atomicCAS(p.err, 0, 2 | (me << 4) | (mode << 8) | (kb << 12) | ((int)blockIdx.x << 20));
          *s_fail = 1;
          break;
        }
        ptx::tc_fence_after();
        const uint64_t da = d_a0 + (uint64_t)((uint32_t)st * stage16), db = da + ab16;
        if (PAIR) {
          ptx::umma_bf16_pair_if(on, d_acc, da, db, idesc, acc);
#pragma unroll
          for (int k = 1; k < 4; ++k) ptx::umma_bf16_pair_if(on, d_acc, da + 2 * k, db + 2 * k, idesc, 1);
          ptx::umma_commit_pair_if(on, empty_mine + (uint32_t)st * 8u);
          ptx::umma_commit_pair_if(on, empty_peer + (uint32_t)st * 8u);
        } else {
          ptx::umma_bf16_if(on, d_acc, da, db, idesc, acc);
#pragma unroll
          for (int k = 1; k < 4; ++k) ptx::umma_bf16_if(on, d_acc, da + 2 * k, db + 2 * k, idesc, 1);
          ptx::umma_commit_if(on, &empty[st]);
        }
        acc = 1;
      }
      // arrives when every UMMA above has finished (also on the failure path)
      if (PAIR) {
        ptx::umma_commit_pair_if(on, ptx::smem_u32(accum));
        ptx::umma_commit_pair_if(on, ptx::map_to_cta(ptx::smem_u32(accum), 1u));
      } else {
        ptx::umma_commit_if(on, accum);
      }
    }
  } else {
    // ---------------- epilogue: 4 EPI_GROUPS warps; a thread owns one output row and every EPI_GROUPS-th 16-column chunk ----------------
    // (the epilogue of a tile is a chain of long-latency steps - TMEM load, special functions, stores -
    // so it is spread over as many warps as there are chunks in the common 64-column tile)
    // Everything that does not depend on the accumulator is fetched while the main loop runs:
    // per-column constants go to shared memory, the thread's residual row (or, for a left-context
    // row, the carried row) goes to registers.
    const int et = threadIdx.x - 128;
    if (et < BN) s_bias[et] = p.bias[n0 + et];   // BN <= 192 < EPI_THREADS
    ptx::pdl_wait();                              // slot table, residual and carry rows are upstream data
    if (p.tau != nullptr && et < 2 * BN) {      // conv blocks (BN <= 64): the timestep bias of each of the tile's two slots
      const int sl = et / BN, c = et - sl * BN, ts = m0 / SLOT_ROWS + sl;
      s_tau[sl * 64 + c] = ts < p.n_slots ? p.tau[p.slots[ts].tau_off + n0 + c] : 0.f;
    }
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int cg = (warp - 4) >> 2;               // which chunks of the row: chunk index % EPI_GROUPS == cg
    const int r = m0 + q * 32 + lane;             // row in slot layout (without GUARD)
    const int slot = r / SLOT_ROWS, rho = r % SLOT_ROWS;
    const SlotInfo si = slot < p.n_slots ? p.slots[slot] : SlotInfo{0, 0, 0, 0, nullptr, nullptr, nullptr, nullptr, 0, 0, 0, 0, 0, 0, 0};
    const bool in_range = si.T > 0;               // (a slot without frames - a hole in a wavefront - is left alone)
    const int f = rho - HALO;
    const bool do_halo = p.halo_off >= 0;
    const bool has_resid = mode == MODE_CONV || mode == MODE_OPROJ;
    const long long grow = (long long)(GUARD + r);
    bf16* carry = do_halo && in_range ? si.halo + p.halo_off : nullptr;
    // pre[2k], pre[2k+1]: the 16 bf16 of this thread's k-th chunk (columns n0 + 16 (EPI_GROUPS k + cg) ..);
    // the GEMMs with a residual or carried rows have at most 64 columns per tile
    constexpr int PRE_CHUNKS = 4 / EPI_GROUPS;
    uint4 pre[2 * PRE_CHUNKS];
#pragma unroll
    for (int j = 0; j < 2 * PRE_CHUNKS; ++j) pre[j] = make_uint4(0u, 0u, 0u, 0u);
    {
      const bf16* src = nullptr;
      if (in_range && f >= 0 && f < si.T && has_resid) src = p.resid + grow * p.ld + n0;
      else if (in_range && rho < HALO && do_halo) src = carry + rho * p.C + n0;
      if (src != nullptr) {
#pragma unroll
        for (int k = 0; k < PRE_CHUNKS; ++k) {
          if (16 * (EPI_GROUPS * k + cg) < BN) {
            pre[2 * k] = *reinterpret_cast<const uint4*>(src + 16 * (EPI_GROUPS * k + cg));
            pre[2 * k + 1] = *reinterpret_cast<const uint4*>(src + 16 * (EPI_GROUPS * k + cg) + 8);
          }
        }
      }
    }
    // row scale 1 / rms of the normalised operand: chunk partials in ascending order
    float rs = 1.f;
    if (p.ssq_in != nullptr) {
      float ss = 0.f;
      if (in_range && f >= 0 && f < si.T) {
        const int n_parts = p.C >> 4;
        for (int j = 0; j < n_parts; ++j) ss += p.ssq_in[(long long)j * p.ssq_ld + r];
      }
      rs = rsqrtf(ss * p.inv_C + p.eps);
    }
    // constants visible to all epilogue threads; every read of the carry has been performed
    // before any thread below overwrites carry rows
    ptx::named_bar_sync(1, EPI_THREADS);

    const bool got = ptx::mbar_wait_relaxed(accum, 0);
    if (PAIR) ptx::cluster_wait();   // (long complete; a thread waits once between its two arrivals)
    ptx::tc_fence_after();
    if (!got) atomicCAS(p.err, 0, 3 | (mode << 8));
    const bool slot_ok = in_range && got && *s_fail == 0;
    const float* tau_s = s_tau + ((q >> 1) & 1) * 64;   // rows 64.. of the tile are its second slot
    const bool is_halo = slot_ok && rho < HALO;
    const bool is_chunk = slot_ok && f >= 0 && f < si.T;
    const int new_row = rho - si.Tc;              // carry row this thread's value moves to (the carry follows the committed frames)
    const bool carry_wr = do_halo && (is_halo || is_chunk) && new_row >= 0 && new_row < HALO;

    // PAIR: tensor memory is freed for both CTAs at once, so each thread reports its LAST accumulator load
    // to the cluster barrier as soon as it has happened; the barrier's latency (about 1500 cycles) then runs
    // under the arithmetic and the stores that follow, and the freeing warp finds it complete.
    const int last_kk = (BN - 16 * cg - 1) / (16 * EPI_GROUPS);   // (BN > 16 cg for every chunk group of a paired GEMM)
    // (in the generic kernel, the one of small batches, the loop stays a loop: three unrolled copies of the epilogue
    // body are code that has to come through the instruction cache at every one of their short launches - cfg3 1.371 ->
    // 1.359 ms per chunk; the kernels of a role keep them: a QKV thread overlaps its three chunks, 1.911 against 1.926)
#pragma unroll(MODE_T >= 0 ? MAX_BN / (16 * EPI_GROUPS) : 1)
    for (int kk = 0; kk < MAX_BN / (16 * EPI_GROUPS); ++kk) {
      const int ch = EPI_GROUPS * kk + cg;
      const int c0 = ch * 16;
      if (c0 >= BN) break;
      float acc[16];
      // The kernel of the conv role has the registers for taps 0 and 1 of both issuers behind ONE wait (the generic
      // kernel spills with it); tap 2 fetched ahead of the exchange barrier as well measured slower (1.908 against 1.901).
      constexpr bool FOUR_LOADS = MODE_T == MODE_CONV && BN_T > 0;
      float z01[16];
      if (FOUR_LOADS) {
        const uint32_t lanes = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t ra[32], rb[32];
        ptx::tmem_ld16x2_issue(lanes + (uint32_t)c0, lanes + acc2_off + (uint32_t)c0, ra);
        ptx::tmem_ld16x2_issue(lanes + (uint32_t)(BN + c0), lanes + acc2_off + (uint32_t)(BN + c0), rb);
        ptx::tmem_ld_wait32(ra);
        ptx::tmem_ld_wait32(rb);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          acc[i] = __uint_as_float(ra[i]) + __uint_as_float(ra[16 + i]);
          z01[i] = __uint_as_float(rb[i]) + __uint_as_float(rb[16 + i]);
        }
      } else if (n_iss == 2) {   // even blocks + odd blocks, always in this order
        float acc2[16];
        ptx::tmem_ld16x2(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, tmem_base + ((uint32_t)(q * 32) << 16) + acc2_off + (uint32_t)c0,
                         acc, acc2);
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] += acc2[i];
      } else {
        ptx::tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, acc);
      }
      if (n_taps == 3) {
        // conv block: acc holds tap 0's product for this row; y[r] = Z_0[r - shift_0] + Z_1[r - shift_1] + Z_2[r].
        // A row is a TMEM lane, which a thread cannot change, so the shifted rows go through shared memory
        // (the operand stages are idle by now).  Shifts never leave the slot for the rows that are
        // stored (<= 8 left-context rows precede the chunk).
        float z[16];
        const uint32_t lanes = tmem_base + ((uint32_t)(q * 32) << 16);
        if (FOUR_LOADS) {
#pragma unroll
          for (int i = 0; i < 16; ++i) z[i] = z01[i];
        } else if (n_iss == 2) {
          float t[16];
          ptx::tmem_ld16x2(lanes + (uint32_t)(BN + c0), lanes + acc2_off + (uint32_t)(BN + c0), z, t);
#pragma unroll
          for (int i = 0; i < 16; ++i) z[i] += t[i];
        } else {
          ptx::tmem_ld16(lanes + (uint32_t)(BN + c0), z);
        }
        // exchange area of this chunk group: Z_0 then Z_1, each [4 float4 columns][128 rows] (a warp's 32 rows
        // are 512 contiguous bytes, shifted or not: no bank conflicts); conv tiles have <= 64 columns, so kk = 0
        float4* xz = reinterpret_cast<float4*>(smem) + cg * (2 * 4 * TILE_M);
        const int row_t = q * 32 + lane;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          xz[j * TILE_M + row_t] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          xz[(4 + j) * TILE_M + row_t] = make_float4(z[4 * j], z[4 * j + 1], z[4 * j + 2], z[4 * j + 3]);
        }
        ptx::named_bar_sync(2 + cg, 128);   // the four warps that own this chunk
        const int r0 = max(row_t - p.shift[0], 0), r1 = max(row_t - p.shift[1], 0);   // (row 0 of a tile is a left-context row)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 a0 = xz[j * TILE_M + r0], a1 = xz[(4 + j) * TILE_M + r1];
          acc[4 * j] = a0.x + a1.x;
          acc[4 * j + 1] = a0.y + a1.y;
          acc[4 * j + 2] = a0.z + a1.z;
          acc[4 * j + 3] = a0.w + a1.w;
        }
        if (n_iss == 2) {
          float t[16];
          ptx::tmem_ld16x2(lanes + (uint32_t)(2 * BN + c0), lanes + acc2_off + (uint32_t)(2 * BN + c0), z, t);
#pragma unroll
          for (int i = 0; i < 16; ++i) z[i] += t[i];
        } else {
          ptx::tmem_ld16(lanes + (uint32_t)(2 * BN + c0), z);
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] += z[i];
      }
      if (PAIR && kk == last_kk) {
        ptx::tc_fence_before();
        ptx::cluster_arrive();
      }
      const int n = n0 + c0;
#pragma unroll
      for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], rs, s_bias[c0 + i]);
      if (mode == MODE_OUT) {
        if (p.cfg_w > 0.f) {
          // guided step: rows 64.. of the tile are the unconditional pass of the stream in rows 0..63; they hand
          // their velocity over through shared memory and the conditional rows form (1 + w) v_c - w v_u
          // (16-column tiles: this chunk group's four warps are the only ones here)
          float4* xv4 = reinterpret_cast<float4*>(smem);
          if (q >= 2) {
#pragma unroll
            for (int j = 0; j < 4; ++j) xv4[j * 64 + (q - 2) * 32 + lane] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          }
          ptx::named_bar_sync(2 + cg, 128);
          if (q < 2) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float4 u = xv4[j * 64 + q * 32 + lane];
              acc[4 * j] = fmaf(1.f + p.cfg_w, acc[4 * j], -p.cfg_w * u.x);
              acc[4 * j + 1] = fmaf(1.f + p.cfg_w, acc[4 * j + 1], -p.cfg_w * u.y);
              acc[4 * j + 2] = fmaf(1.f + p.cfg_w, acc[4 * j + 2], -p.cfg_w * u.z);
              acc[4 * j + 3] = fmaf(1.f + p.cfg_w, acc[4 * j + 3], -p.cfg_w * u.w);
            }
          }
        }
        if (is_chunk && si.pass == 0) {
          float* xs = p.xstate + (long long)r * p.mel + n;
          float xv[16];
#pragma unroll
          for (int i = 0; i < 16; i += 4) {
            const float4 t = *reinterpret_cast<const float4*>(xs + i);
            xv[i] = t.x; xv[i + 1] = t.y; xv[i + 2] = t.z; xv[i + 3] = t.w;
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) xv[i] = xv[i] + acc[i] * p.inv_n;
#pragma unroll
          for (int i = 0; i < 16; i += 4)
            *reinterpret_cast<float4*>(xs + i) = make_float4(xv[i], xv[i + 1], xv[i + 2], xv[i + 3]);
          uint4 a, b;
          pack16_bf16(xv, a, b);
          store16(p.ain + grow * p.ld_ain + n, a, b);
          if (p.cfg_w > 0.f) store16(p.ain + (grow + SLOT_ROWS) * p.ld_ain + n, a, b);   // the unconditional pass starts from the same x
          if ((p.last_step || (si.flags & SLOT_LAST)) && f < si.Tc) {
            float* o = si.out + (long long)f * p.mel + n;
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              *reinterpret_cast<float4*>(o + i) = make_float4(xv[i], xv[i + 1], xv[i + 2], xv[i + 3]);
          }
        }
        continue;
      }
      if (mode == MODE_QKV) {
        if (is_chunk) {
          uint4 a, b;
          pack16_bf16(acc, a, b);
          const int which = (n >= p.C) + (n >= 2 * p.C), col = n - which * p.C;   // 0: Q, 1: K, 2: V (no division)
          if (which == 0) {
            store16(p.q_out + grow * p.ld + col, a, b);
          } else {
            // the chunk's first tp frames complete the prompt, the others go to the history ring behind it
            const int tp = min(si.T, p.P - si.n_prompt0);
            int row;
            if (f < tp) {
              row = si.n_prompt0 + f;
            } else {
              row = si.kv_head + f - tp;
              if (row >= p.Rk) row -= p.Rk;
              row += p.P;
            }
            const int hh = col >> p.dh_shift, wi = col - (hh << p.dh_shift);
            // head_dim 64: a K / V row is stored with its 16-byte chunks in the order of the swizzled shared-memory row
            // that the attention kernel copies it to, chunk c at position c ^ (row & 7).  The two chunks of this
            // thread stay inside their 32 bytes, swapped for odd rows.
            const int wp = p.dh_shift == 6 ? ((((wi >> 3) ^ (row & 7)) & ~1) << 3) : wi;
            const bool swap = p.dh_shift == 6 && (row & 1);
            store16(si.kv + p.kv_off + (long long)(which - 1) * (p.P + p.Rk) * p.C + (long long)hh * p.kv_hs + (long long)row * p.kv_rs + wp,
                    swap ? b : a, swap ? a : b);
          }
        }
        continue;
      }
      // modes with a bf16 activation output: INPROJ, CONV, OPROJ (BN <= 64, so kk < 2)
      uint4 va = pre[(2 * kk) % (2 * PRE_CHUNKS)], vb = pre[(2 * kk + 1) % (2 * PRE_CHUNKS)];
      if (!is_halo) {
        if (has_resid) {
          const uint32_t w[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
          if (mode == MODE_CONV) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              acc[2 * i] = __uint_as_float(w[i] << 16) + silu_f(acc[2 * i] + tau_s[c0 + 2 * i]);
              acc[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u) + silu_f(acc[2 * i + 1] + tau_s[c0 + 2 * i + 1]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              acc[2 * i] += __uint_as_float(w[i] << 16);
              acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
            }
          }
        }
        pack16_bf16(acc, va, vb);
      }
      // chunk rows store y; left-context rows hand the carried rows to the consumer of `out`
      if (is_chunk || (is_halo && do_halo)) store16(p.out + grow * p.ld + n, va, vb);
      if (p.ssq_out != nullptr && in_range) {   // sum of squares of the 16 stored values, fixed order
        float ss = 0.f;
        if (is_chunk) {
          const uint32_t w[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
            ss = fmaf(lo, lo, ss);
            ss = fmaf(hi, hi, ss);
          }
        }
        p.ssq_out[(long long)(n >> 4) * p.ssq_ld + r] = ss;
      }
      // shift the carry by T frames: [old carry | chunk] -> its last 8 rows
      if (carry_wr) store16(carry + new_row * p.C + n, va, vb);
    }
  }
  if (PAIR) {
    // Nothing of a CTA is touched by its partner after its own waits have returned (its copies count on the
    // even CTA's barriers, which that CTA waits for; the UMMAs that read its shared memory are complete when
    // its accumulator barrier fires), so a CTA may leave as soon as tensor memory can be freed: when every
    // thread of the pair has arrived, the epilogue threads having done so after their last accumulator load.
    // (warps that have not waited on the first phase yet do so now)
    if (warp < 4 && !(((warp & 1) == 0 && pair_rank != 0) || ((warp & 1) == 1 && (warp >> 1) < n_iss && pair_rank == 0))) ptx::cluster_wait();
    if (warp < 4) ptx::cluster_arrive();
    if (warp == 1) {
      ptx::cluster_wait();
      ptx::tc_fence_after();
      ptx::tmem_dealloc_pair(tmem_base, tmem_cols);
    }
  } else {
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, tmem_cols);
  }
}

// ---- small kernels ---------------------------------------------------------------------------

// Waits on a barrier that nothing completes; the bounded wait must return false.  result: 1 = gave
// up as it should, 2 = claimed success.
__global__ void bounded_wait_selftest_kernel(uint32_t max_polls, int* result) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
    const bool got = ptx::mbar_wait_limit(&bar, 0, max_polls);
    *result = got ? 2 : 1;
  }
}

__global__ void set_slots_kernel(const SlotSet set, SlotInfo* dst) {
  ptx::pdl_launch();
  const int i = threadIdx.x;
  if (i < set.count) dst[set.first + i] = set.s[i];
}

// feats [T][2 mel] (or [T][mel] when the noise is drawn here) -> Euler state x_0 (fp32) and the bf16
// input-projection operand [x_0 | mu].  Device noise: the draw of (frame t, channels 4g..4g+3) is Philox at
// counter (t, g, stream) under the model's seed - the offset is the stream's frame clock, so a replayed graph
// draws what direct launches would, and a look-ahead frame draws the same noise when it is presented again.
__global__ void flow_prep_kernel(const SlotInfo* slots, int mel, float* xstate, bf16* ain, int ld_ain, uint32_t seed_lo, uint32_t seed_hi) {
  ptx::pdl_launch();
  ptx::pdl_wait();
  const SlotInfo si = slots[blockIdx.x];
  if (!(si.flags & SLOT_FIRST)) return;      // (wavefront: this slot's chunk is past its first Euler step)
  const bool draw = (seed_lo | seed_hi) != 0u;
  const int fw = draw ? mel : 2 * mel;       // width of a row of feats
  for (int i = threadIdx.x; i < si.T * (mel / 4); i += blockDim.x) {
    const int f = i / (mel / 4), g = i - f * (mel / 4);
    const long long r = (long long)blockIdx.x * SLOT_ROWS + HALO + f;
    float x0[4];
    if (draw) {
      const unsigned long long t = (unsigned long long)(si.frame0 + f);
      uint32_t w[4];
      philox4x32_10((uint32_t)t, (uint32_t)(t >> 32), (uint32_t)g, (uint32_t)si.rng_id, seed_lo, seed_hi, w);
      normals4(w, x0);
    } else {
      const float4 v = *reinterpret_cast<const float4*>(si.feats + (long long)f * fw + mel + 4 * g);
      x0[0] = v.x; x0[1] = v.y; x0[2] = v.z; x0[3] = v.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = 4 * g + j;
      const float mu = si.pass == 0 ? si.feats[(long long)f * fw + c] : 0.f;
      xstate[r * mel + c] = x0[j];
      ain[(GUARD + r) * ld_ain + c] = __float2bfloat16_rn(x0[j]);
      ain[(GUARD + r) * ld_ain + mel + c] = __float2bfloat16_rn(mu);
    }
  }
}

// u = bf16(x * rsqrt(mean(x^2) + eps)), one warp per chunk row: the normalised activation as a stored, rounded
// tensor (DC_OPT_ROUNDED_NORM) instead of a row scale folded into the consuming GEMM's accumulator.  The row
// statistic is the one the producing GEMM left (partial sums of squares per 16-column chunk, added in chunk
// order), so both forms of the norm use the same 1 / rms.
__global__ void flow_rmsnorm_kernel(const SlotInfo* slots, int n_slots, const bf16* x, bf16* u, int C, const float* ssq, long long ssq_ld,
                                    float inv_C, float eps) {
  ptx::pdl_launch();
  ptx::pdl_wait();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int slot = warp / SLOT_ROWS, rho = warp % SLOT_ROWS;
  if (slot >= n_slots) return;
  const int f = rho - HALO;
  if (f < 0 || f >= slots[slot].T) return;
  float ss = 0.f;
  for (int j = 0; j < (C >> 4); ++j) ss += ssq[(long long)j * ssq_ld + warp];
  const float rs = rsqrtf(ss * inv_C + eps);
  const long long off = (long long)(GUARD + warp) * C;
  for (int c = lane * 8; c < C; c += 256) {
    const uint4 v = *reinterpret_cast<const uint4*>(x + off + c);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(w[i] << 16) * rs, __uint_as_float(w[i] & 0xFFFF0000u) * rs);
      o[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(u + off + c) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---- chunk-causal attention with the K/V carry ---------------------------------------------------
// One CTA per (stream slot, head), two CTAs per SM.  Queries: the T <= 56 chunk frames, held TWICE
// in the 128 UMMA rows (row 64 + i repeats row i), so that S has a copy of every query row in both
// halves of tensor memory: a warp can only read the 32 lanes of its own SM sub-partition, and with
// the copy the softmax work spreads over all four sub-partitions (special-function throughput is
// what bounds it) instead of the two that own lanes 0..63.  Keys/values: the kv_len carried frames
// followed by the chunk's own T frames, streamed in place from the stream's ring in blocks of 128
// keys with 128-bit cp.async loads (the ring may wrap; nothing is compacted or copied in global
// memory) through a two-stage shared-memory ring.
//
// Warp roles (8 warps): warps 0..3 = softmax (thread = (query row, half of the block's 128 key
// columns); warps 0,1 read lanes 0..63 and own key columns 0..63, warps 2,3 read the copy in lanes
// 64..127 and own key columns 64..127); warp 4 = UMMA issuer; warps 5,6 = Q and K loaders, warp 7 =
// V loader.
// Per key block: S = Q K^T on tcgen05 (accumulator in TMEM) -> the softmax threads read their
// columns, e = exp2(scale*S - m) with a running reference m that is only raised when the block
// maximum exceeds it by more than 2^8 (then O and the row sum are rescaled once), row sum from the
// unrounded e, P = bf16(e) into shared memory (64 rows; the UMMA's rows 64..127 of P and O are
// never read back) -> O += P V on tcgen05 (V is the MN-major operand).  O lives in lanes 0..63, so
// warps 0,1 rescale it and write the result.
constexpr int ATT_THREADS = 256;
constexpr int ATT_KB = 128;             // keys per block
constexpr int ATT_STAGES = 2;
constexpr int ATT_TMEM_COLS = 256;      // S (128 columns) + O (64 columns); two CTAs share the SM's 512
constexpr int ATT_K_LOADERS = 64;       // warps 5 and 6: Q, then the K blocks
constexpr int ATT_V_LOADERS = 32;       // warp 7: the V blocks
constexpr int ATT_Q_BYTES = 128 * 128;  // 64 query rows, twice
constexpr int ATT_P_BYTES = 2 * 64 * 128;   // one P buffer: 64 rows x 128 keys; there are two
constexpr int ATT_STAGE_BYTES = 2 * ATT_KB * 128;   // K block + V block
constexpr int ATT_BAR_BYTES = 1024;        // 14 barriers, TMEM slot, softmax exchange (512 B)
// Two CTAs per SM leave 113 KB each: the tiles take 112 KB, so there is no room for alignment slack.
// The dynamic shared memory is declared 1024-byte aligned (the swizzled tiles need it) and the kernel
// checks the address it got.
constexpr size_t ATT_SMEM = ATT_Q_BYTES + 2 * ATT_P_BYTES + ATT_STAGES * ATT_STAGE_BYTES + ATT_BAR_BYTES;
static_assert(ATT_SMEM <= 113 * 1024 + 1024, "two attention CTAs must fit one SM");
constexpr float ATT_RESCALE_LOG2 = 8.0f;

struct AttnParams {
  const SlotInfo* slots;
  const bf16*     q;          // [GUARD + rows][ld]
  bf16*           o;          // [GUARD + rows][ld]
  int             ld;
  int             dh;         // 32 or 64 (smem rows are padded to 64 columns)
  long long       kv_off;     // element offset of this (step, layer)'s K ring inside SlotInfo::kv
  int             kv_rs, kv_hs;   // K/V planes: elements between a head's consecutive rows / between heads
  int             Rk, C;
  int             P;          // prompt rows in front of the ring
  float           scale_log2e;  // log2(e) / sqrt(dh)
  int*            err;
  int             empty;      // measurement only: the kernel returns at once (the cost of the bare stage boundary)
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(dst)), "l"(src) : "memory");
}

// PROMPT = false: the carry is a plain window (no prompt rows); a separate instantiation, because this kernel sits at its
// register limit and the copy loops of its loader warps pace it.
// BULK (no prompt rows, head_dim 64): a head's K / V rows are 128 contiguous bytes each, stored with their 16-byte
// chunks already in the order of the swizzled shared-memory row they will occupy (chunk c of plane row r at
// position c ^ (r & 7)), and the ring is walked from the 8-row boundary below the attended interval, so that a block
// of 128 keys is one flat span of 16 KB (two at the ring's wrap) with shared-memory row == plane row (mod 8): ONE thread
// fetches it with one or two untiled bulk copies that complete on the stage's barrier.  The up to seven keys in front
// of the interval are masked like the padding behind it.  Without BULK the loader warps copy 16 bytes per thread and
// instruction (about 2,800 cycles of issue per block and warp).
template <bool PROMPT, bool BULK>
__global__ void __launch_bounds__(ATT_THREADS, 2) flow_attn_kernel(const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t att_smem_raw[];
  uint8_t* smem = att_smem_raw;
  if (p.empty) {
    ptx::pdl_launch();
    ptx::pdl_wait();
    return;
  }
  if ((ptx::smem_u32(smem) & 1023u) != 0u) {   // would corrupt the swizzled tiles: refuse (uniform for the CTA)
    if (threadIdx.x == 0) atomicExch(p.err, 14);
    return;
  }
  uint8_t* sQ = smem;
  uint8_t* sP = sQ + ATT_Q_BYTES;                    // buffer b & 1 at + ATT_P_BYTES (b & 1); tile t (keys 64 t .. of the block) at + 8192 t
  uint8_t* ring = sP + 2 * ATT_P_BYTES;
  // K and V have their own two-stage rings: a K stage is free as soon as S of its block has been
  // computed, long before the V stage of the same block (free after P V), so K runs further ahead.
  uint64_t* full_k = reinterpret_cast<uint64_t*>(ring + ATT_STAGES * ATT_STAGE_BYTES);   // [ATT_STAGES] each
  uint64_t* empty_k = full_k + ATT_STAGES;
  uint64_t* full_v = empty_k + ATT_STAGES;
  uint64_t* empty_v = full_v + ATT_STAGES;
  uint64_t* bar_s = empty_v + ATT_STAGES;
  // P and "P V done" have one barrier per P buffer (block parity): with a single barrier a waiter
  // that falls a whole block behind could not tell phase b from phase b + 2.
  uint64_t* bar_p = bar_s + 1;          // [2]: all softmax threads have written P(b) into buffer b & 1
  uint64_t* bar_pv = bar_p + 2;         // [2]: P(b) V(b) has been accumulated: buffer b & 1 is free, O holds blocks <= b
  uint64_t* bar_sfree = bar_pv + 2;     // every softmax thread has copied its S columns to registers
  uint64_t* bar_q = bar_sfree + 1;      // BULK: Q has landed (without BULK it is published with the first K block)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_sfree + 2);
  float* s_x = reinterpret_cast<float*>(tmem_slot + 2);   // [2][64] exchange between the two column halves

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slot = blockIdx.x, head = blockIdx.y;
  const int chunks = p.dh >> 3;             // 16-byte chunks per head row

  if (tid == 0) {
    for (int i = 0; i < ATT_STAGES; ++i) {
      ptx::mbar_init(&full_k[i], BULK ? 1 : ATT_K_LOADERS);
      ptx::mbar_init(&empty_k[i], 1);
      ptx::mbar_init(&full_v[i], BULK ? 1 : ATT_V_LOADERS);
      ptx::mbar_init(&empty_v[i], 1);
    }
    ptx::mbar_init(bar_s, 1);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&bar_p[i], 128);
      ptx::mbar_init(&bar_pv[i], 1);
    }
    ptx::mbar_init(bar_sfree, 128);
    ptx::mbar_init(bar_q, ATT_K_LOADERS);
    ptx::fence_barrier_init();
  }
  if (warp == 4) ptx::tmem_alloc(tmem_slot, ATT_TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch();
  // Q and the chunk's appended K/V rows come from the kernel before this one.  The slot table and the CARRIED K/V
  // rows do not (the table is written by the first kernel of the step, which has completed before any projection
  // starts; carried rows by earlier steps), so the loader warps fetch the leading all-carried key blocks first
  // and wait afterwards.
  if (warp < 5) ptx::pdl_wait();
  const SlotInfo si = p.slots[slot];
  // attended keys, in this order: the prompt rows (with the chunk's own prompt frames, already appended), then
  // the carried history and the chunk's history frames, a circular interval of the ring behind the prompt rows
  const int T = si.T;
  const int n_prompt = PROMPT ? si.n_prompt0 + min(T, p.P - si.n_prompt0) : 0;
  const int L0 = PROMPT ? n_prompt + si.kv_len + (T - (n_prompt - si.n_prompt0)) : si.kv_len + T;
  int ring_start = si.kv_head - si.kv_len;      // ring row of the oldest attended history frame
  if (ring_start < 0) ring_start += p.Rk;
  const int phi = BULK ? (ring_start & 7) : 0;  // BULK: keys 0 .. phi - 1 are the rows between the 8-row boundary and the interval
  const int L = L0 + phi;
  const int nkb = (L + ATT_KB - 1) / ATT_KB;

  if (T == 0) {
    // a slot without frames (a hole in a wavefront): nothing to do but to release tensor memory below
  } else if (BULK && warp >= 5) {
    // ---------------- loaders, bulk copies: lane 0 of warp 5 fetches the K blocks, lane 0 of warp 7 the V blocks;
    // warps 5 and 6 copy Q (64 rows of the projection's output, each held twice) ----------------
    const bool is_k = warp != 7;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    const bf16* src0 = si.kv + p.kv_off + (long long)head * p.kv_hs + (is_k ? 0 : (long long)p.Rk * p.C);
    uint64_t* full = is_k ? full_k : full_v;
    uint64_t* empty = is_k ? empty_k : empty_v;
    const int row0 = ring_start - phi;                     // a multiple of 8 (the ring has a multiple of 8 rows)
    const int n_early = min(min((si.kv_len + phi) / ATT_KB, ATT_STAGES), nkb);   // blocks of carried rows only (< nkb: the chunk's rows come last)
    bool ok = true;
    auto fetch = [&](int b) {                               // warps 5 and 7, all lanes (lane 0 issues)
      const int st = b % ATT_STAGES;
      if (b >= ATT_STAGES && ok && !ptx::mbar_wait_relaxed(&empty[st], ((b / ATT_STAGES) - 1) & 1)) {
        ok = false;
        atomicExch(p.err, 4);
      }
      uint8_t* dstb = ring + st * ATT_STAGE_BYTES + (is_k ? 0 : ATT_KB * 128);
      const int n = min(ATT_KB, L - b * ATT_KB);            // key rows of this block
      if (!is_k && n < ATT_KB) {
        // the P V product reads whole 16-row steps: the rows behind the last key must be finite (their weights are 0)
        const int n16 = min(ATT_KB, (n + 15) & ~15);
        for (int i = lane; i < (n16 - n) * 8; i += 32) *reinterpret_cast<uint4*>(dstb + n * 128 + i * 16) = zero;
        ptx::fence_proxy_async_smem();
        __syncwarp();
      }
      if (lane == 0) {
        int rr = row0 + b * ATT_KB;
        while (rr >= p.Rk) rr -= p.Rk;
        const int n1 = min(n, p.Rk - rr);
        ptx::mbar_expect_tx(&full[st], (uint32_t)n * 128u);
        ptx::bulk_load(dstb, src0 + (long long)rr * 64, (uint32_t)n1 * 128u, &full[st]);
        if (n1 < n) ptx::bulk_load(dstb + n1 * 128, src0, (uint32_t)(n - n1) * 128u, &full[st]);
      }
    };
    if (warp != 6)
      for (int b = 0; b < n_early; ++b) fetch(b);           // (b < ATT_STAGES: no stage to wait for)
    ptx::pdl_wait();                                        // Q and the chunk's own K / V rows are the projection's output
    if (is_k) {
      const int lt = (warp == 6 ? 32 : 0) + lane;
      const bf16* qbase = p.q + (long long)(GUARD + slot * SLOT_ROWS + HALO) * p.ld + head * 64;
      for (int i = lt; i < 128 * 8; i += ATT_K_LOADERS) {
        const int row = i >> 3, j = i & 7, qrow = row & 63;   // rows 64.. repeat rows 0..
        uint8_t* dst = sQ + row * 128 + ((j ^ (row & 7)) << 4);
        if (qrow < T) cp_async16(dst, qbase + (long long)qrow * p.ld + j * 8);
        else *reinterpret_cast<uint4*>(dst) = zero;
      }
      asm volatile("cp.async.wait_all;" ::: "memory");
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(bar_q);
    }
    if (warp != 6)
      for (int b = n_early; b < nkb; ++b) fetch(b);
  } else if (warp >= 5) {
    // ---------------- loaders ----------------
    const bool is_k = warp != 7;
    const int nl = is_k ? ATT_K_LOADERS : ATT_V_LOADERS;
    const int lt = (warp == 6 ? 32 : 0) + lane;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    const bf16* src0 = si.kv + p.kv_off + (long long)head * p.kv_hs + (is_k ? 0 : (long long)((PROMPT ? p.P : 0) + p.Rk) * p.C);
    const int rs = p.kv_rs;
    uint64_t* full = is_k ? full_k : full_v;
    uint64_t* empty = is_k ? empty_k : empty_v;
    const int start = ring_start;
    // head_dim 64: chunk j of plane row rr is stored at position j ^ (rr & 7) (see BULK); head_dim 32 rows are stored plainly
    const int perm = p.dh == 64 ? 7 : 0;
    auto issue_block = [&](int b) {
      uint8_t* dstb = ring + (b % ATT_STAGES) * ATT_STAGE_BYTES + (is_k ? 0 : ATT_KB * 128);
      if (!PROMPT) {
        for (int i = lt; i < ATT_KB * 8; i += nl) {
          const int row = i >> 3, j = i & 7;
          const int key = b * ATT_KB + row;
          const int off = row * 128 + ((j ^ (row & 7)) << 4);
          if (key < L && j < chunks) {
            int rr = start + key;
            if (rr >= p.Rk) rr -= p.Rk;
            cp_async16(dstb + off, src0 + (long long)rr * rs + ((j ^ (rr & perm)) << 3));
          } else {
            *reinterpret_cast<uint4*>(dstb + off) = zero;   // for V: 0 * garbage must not poison O
          }
        }
      } else if ((b + 1) * ATT_KB <= n_prompt) {
        // a block of prompt rows only: row index = key
        for (int i = lt; i < ATT_KB * 8; i += nl) {
          const int row = i >> 3, j = i & 7;
          const int off = row * 128 + ((j ^ (row & 7)) << 4);
          if (j < chunks) cp_async16(dstb + off, src0 + (long long)(b * ATT_KB + row) * rs + ((j ^ (row & perm)) << 3));
          else *reinterpret_cast<uint4*>(dstb + off) = zero;
        }
      } else {
        // the block where the prompt rows end and the ring behind them begins (or ring rows only)
        for (int i = lt; i < ATT_KB * 8; i += nl) {
          const int row = i >> 3, j = i & 7;
          const int key = b * ATT_KB + row;
          const int off = row * 128 + ((j ^ (row & 7)) << 4);
          if (key < L && j < chunks) {
            int rr = key;                            // a prompt row, or ...
            if (key >= n_prompt) {                   // ... a ring row behind the prompt rows
              rr = start + key - n_prompt;
              if (rr >= p.Rk) rr -= p.Rk;
              rr += p.P;
            }
            cp_async16(dstb + off, src0 + (long long)rr * rs + ((j ^ (rr & perm)) << 3));
          } else {
            *reinterpret_cast<uint4*>(dstb + off) = zero;
          }
        }
      }
    };
    // keys [0, carried) were appended by earlier steps: the prompt rows already there, and - once the prompt is
    // complete - the retained history behind them
    const int carried = PROMPT ? (n_prompt == si.n_prompt0 ? n_prompt + si.kv_len : si.n_prompt0) : si.kv_len;
    const int n_early = min(min(carried / ATT_KB, ATT_STAGES), nkb);
    for (int b = 0; b < n_early; ++b) issue_block(b);
    ptx::pdl_wait();
    if (is_k) {
      const bf16* qbase = p.q + (long long)(GUARD + slot * SLOT_ROWS + HALO) * p.ld + head * p.dh;
      for (int i = lt; i < 128 * 8; i += nl) {
        const int row = i >> 3, j = i & 7, qrow = row & 63;   // rows 64.. repeat rows 0..
        uint8_t* dst = sQ + row * 128 + ((j ^ (row & 7)) << 4);
        if (qrow < T && j < chunks) cp_async16(dst, qbase + (long long)qrow * p.ld + j * 8);
        else *reinterpret_cast<uint4*>(dst) = zero;
      }
    }
    bool ok = true;
    for (int b = 0; b < nkb; ++b) {
      const int st = b % ATT_STAGES;
      if (b >= 1) {   // the previous block has been issued a whole iteration ago: publish it (block 0 together with Q)
        asm volatile("cp.async.wait_all;" ::: "memory");
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(&full[(b - 1) % ATT_STAGES]);
      }
      if (b < n_early) continue;                                // already in flight
      if (b >= ATT_STAGES && ok && !ptx::mbar_wait_relaxed(&empty[st], ((b / ATT_STAGES) - 1) & 1)) {
        ok = false;
        atomicExch(p.err, 4);
      }
      issue_block(b);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    ptx::fence_proxy_async_smem();
    ptx::mbar_arrive(&full[(nkb - 1) % ATT_STAGES]);
  } else if (warp == 4) {
    // ---------------- UMMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc_s = ptx::umma_idesc_bf16(128, ATT_KB, 0, 0);
      const uint32_t idesc_pv = ptx::umma_idesc_bf16(128, 64, 0, 1);   // B = V, MN-major
      const uint64_t dq = ptx::umma_desc_sw128(ptx::smem_u32(sQ));
      const uint64_t dp = ptx::umma_desc_sw128(ptx::smem_u32(sP));
      bool ok = true;
      // S(b+1) is issued as soon as the softmax threads have copied S(b) out of tensor memory, i.e.
      // before P(b) exists: the tensor pipe computes the next block's scores while the softmax of
      // this block runs, and P V follows when P is ready.
      auto issue_s = [&](int b) {
        const int st = b % ATT_STAGES;
        if (ok && !ptx::mbar_wait(&full_k[st], (b / ATT_STAGES) & 1)) { ok = false; atomicExch(p.err, 5); }
        ptx::tc_fence_after();
        const uint64_t dk = ptx::umma_desc_sw128(ptx::smem_u32(ring + st * ATT_STAGE_BYTES));
#pragma unroll
        for (int k = 0; k < 4; ++k) ptx::umma_bf16(tmem_base, dq + 2 * k, dk + 2 * k, idesc_s, k != 0);
        ptx::umma_commit(bar_s);
        ptx::umma_commit(&empty_k[st]);                  // the K stage is free once S(b) has been computed
      };
      if (BULK && !ptx::mbar_wait(bar_q, 0)) { ok = false; atomicExch(p.err, 12); }
      issue_s(0);
      for (int b = 0; b < nkb; ++b) {
        const int st = b % ATT_STAGES;
        if (b + 1 < nkb) {
          if (ok && !ptx::mbar_wait(bar_sfree, b & 1)) { ok = false; atomicExch(p.err, 10); }
          issue_s(b + 1);
        }
        if (ok && !ptx::mbar_wait(&bar_p[b & 1], (b >> 1) & 1)) { ok = false; atomicExch(p.err, 6); }
        const uint64_t dpb = dp + (uint64_t)((b & 1) * (ATT_P_BYTES >> 4));
        if (ok && !ptx::mbar_wait(&full_v[st], (b / ATT_STAGES) & 1)) { ok = false; atomicExch(p.err, 11); }
        ptx::tc_fence_after();
        const uint64_t dv = ptx::umma_desc_sw128(ptx::smem_u32(ring + st * ATT_STAGE_BYTES + ATT_KB * 128));
        const int valid = L - b * ATT_KB;
        const int ksteps = valid >= ATT_KB ? ATT_KB / 16 : (valid + 15) / 16;
        // P tile k/4 (8 KB apart), 32-byte K steps; V: 16 key rows = 2 KB per step
        if (ksteps == ATT_KB / 16) {
#pragma unroll
          for (int k = 0; k < ATT_KB / 16; ++k)
            ptx::umma_bf16(tmem_base + ATT_KB, dpb + (uint64_t)((k >> 2) * (8192 >> 4) + (k & 3) * 2), dv + (uint64_t)(k * (2048 >> 4)),
                           idesc_pv, (b | k) != 0);
        } else {
          for (int k = 0; k < ksteps; ++k)
            ptx::umma_bf16(tmem_base + ATT_KB, dpb + (uint64_t)((k >> 2) * (8192 >> 4) + (k & 3) * 2), dv + (uint64_t)(k * (2048 >> 4)),
                           idesc_pv, (b | k) != 0);
        }
        ptx::umma_commit(&empty_v[st]);
        ptx::umma_commit(&bar_pv[b & 1]);
      }
    }
  } else {
    // ---------------- softmax: warps 0..3 ----------------
    const int quarter = warp & 1;               // query rows 32*quarter ..
    const int half = warp >> 1;                 // key columns 64*half .. of each block, read from the row copy in lanes 64*half ..
    const int row = quarter * 32 + lane;        // query row
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);   // the lanes this warp may access
    bool ok = true;
    float m_ref = -INFINITY, lsum = 0.f;
    for (int b = 0; b < nkb; ++b) {
      if (ok && !ptx::mbar_wait(bar_s, b & 1)) { ok = false; atomicExch(p.err, 7); }
      ptx::tc_fence_after();
      const int valid = L - b * ATT_KB - half * 64;   // columns of this half that are real keys
      float v[64];
#pragma unroll
      for (int c = 0; c < 4; ++c) ptx::tmem_ld16(lane_addr + (uint32_t)(half * 64 + c * 16), v + 16 * c);
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_sfree);               // S(b) is in registers: the next block's scores may overwrite it
      if (valid < 64) {                          // only the last block has padded key columns
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= valid) v[i] = -INFINITY;
      }
      if (BULK && b == 0 && half == 0) {         // the rows between the 8-row boundary and the attended interval
#pragma unroll
        for (int i = 0; i < 7; ++i)
          if (i < phi) v[i] = -INFINITY;
      }
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; ++i) mx = fmaxf(mx, v[i]);
      s_x[half * 64 + row] = mx * p.scale_log2e;
      ptx::named_bar_sync(2, 128);
      mx = fmaxf(s_x[row], s_x[64 + row]);
      ptx::named_bar_sync(2, 128);   // all have read: the next block (or the row sums below) may overwrite the exchange
      if (b == 0) {
        m_ref = mx;
      } else {
        const bool need = mx > m_ref + ATT_RESCALE_LOG2;
        if (__any_sync(0xffffffffu, need)) {
          // O must hold every earlier block and be quiescent before it is rescaled
          if (ok && !ptx::mbar_wait(&bar_pv[(b - 1) & 1], ((b - 1) >> 1) & 1)) { ok = false; atomicExch(p.err, 8); }
          ptx::tc_fence_after();
          const float alpha = need ? exp2f(m_ref - mx) : 1.0f;
          if (need) m_ref = mx;
          lsum *= alpha;
          if (half == 0) {                        // O rows 0..63 live in lanes 0..63
            for (int c = 0; c < p.dh; c += 16) {
              float o16[16];
              const uint32_t addr = lane_addr + (uint32_t)(ATT_KB + c);
              ptx::tmem_ld16(addr, o16);
#pragma unroll
              for (int i = 0; i < 16; ++i) o16[i] *= alpha;
              ptx::tmem_st16(addr, o16);
            }
          }
          ptx::tc_fence_before();
        }
      }
      if (b >= 2) {   // this block's P buffer was last read by P V of block b - 2
        if (ok && !ptx::mbar_wait(&bar_pv[b & 1], ((b >> 1) - 1) & 1)) { ok = false; atomicExch(p.err, 15); }
      }
      uint8_t* prow = sP + (b & 1) * ATT_P_BYTES + half * 8192 + row * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float e[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          e[i] = ex2_approx(fmaf(v[16 * c + i], p.scale_log2e, -m_ref));
          lsum += e[i];
        }
        uint4 a, bq;
        pack16_bf16(e, a, bq);
        *reinterpret_cast<uint4*>(prow + (((2 * c) ^ (row & 7)) << 4)) = a;
        *reinterpret_cast<uint4*>(prow + (((2 * c + 1) ^ (row & 7)) << 4)) = bq;
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(&bar_p[b & 1]);
    }
    if (ok && !ptx::mbar_wait(&bar_pv[(nkb - 1) & 1], ((nkb - 1) >> 1) & 1)) { ok = false; atomicExch(p.err, 9); }
    ptx::tc_fence_after();
    s_x[half * 64 + row] = lsum;
    ptx::named_bar_sync(2, 128);
    const float inv = 1.0f / (s_x[row] + s_x[64 + row]);
    bf16* orow = p.o + (long long)(GUARD + slot * SLOT_ROWS + HALO + row) * p.ld + head * p.dh;
    for (int c = 0; c < (half == 0 ? p.dh : 0); c += 16) {
      float o16[16];
      ptx::tmem_ld16(lane_addr + (uint32_t)(ATT_KB + c), o16);
      if (row < T && ok) {
#pragma unroll
        for (int i = 0; i < 16; ++i) o16[i] *= inv;
        uint4 a, bq;
        pack16_bf16(o16, a, bq);
        store16(orow + c, a, bq);
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 4) ptx::tmem_dealloc(tmem_base, ATT_TMEM_COLS);
}

// ---- host helpers ----------------------------------------------------------------------------

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}
float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// bf16 row-major [rows][cols] matrix, tiles of box_rows x 64 columns, 128-byte swizzle.
bool make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstr[1] = {cols * sizeof(bf16)};
  cuuint32_t box[2] = {(cuuint32_t)KBLK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t GEMM_SMEM_EXTRA = 1024 + 2 * MAX_STAGES * 8 + 8 + 8 + 2 * MAX_BN * 4 + 64;   // alignment slack + barriers + constants
constexpr size_t GEMM_SMEM_MAX = 200 * 1024;
constexpr int SPECIALISE_FROM_TILES = 8;   // row tiles of a batch from which the GEMMs run as one kernel per role
constexpr size_t GEMM_SMEM_MAX_PAIR = 227 * 1024;   // the opt-in limit of the device: eight 28 KB stages of a CTA pair

}  // namespace

// ---------------------------------------------------------------------------------------------
// engine
// ---------------------------------------------------------------------------------------------

struct GraphEntry {
  cudaGraph_t     graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  cudaGraphNode_t set_node = nullptr;
  int             launches = 0;
  bool            pdl = false;
};

struct FlowModel {
  dc_config cfg;
  int C = 0, mel = 0, Kin = 0, S = 0, rows = 0, Rk = 0, cpa = 0;   // S: slots (streams x passes) of a full batch
  int streams_opened = 0;    // so far: the next stream's random-stream index
  int P = 0;                 // prompt rows in front of every K/V ring
  int n_pass = 1;            // 2 with classifier-free guidance: a stream's conditional and unconditional pass are
                             // adjacent slots, i.e. the two halves of one row tile
  bf16 *Xa = nullptr, *Xb = nullptr, *Q = nullptr, *O = nullptr, *Ain = nullptr;
  bf16 *U = nullptr;         // DC_OPT_ROUNDED_NORM: the normalised activations as a stored bf16 tensor
  float* xstate = nullptr;
  float* ssq = nullptr;      // [C / 16][rows]: per-chunk sums of squares of the rows that feed an RMS norm
  bf16*  wts = nullptr;
  float* fconst = nullptr;   // biases and the timestep-bias table
  SlotInfo* d_slots = nullptr;
  int*   d_err = nullptr;
  CUtensorMap tmAin, tmXa, tmXb, tmO, tmU;
  // weight maps in three tile-width variants v (box rows = N tile): v = 0 wide (64 / 192 / mel), for full
  // batches; v = 1, 2 narrower (32, 16 / 96, 48 / 16), so that a small batch still spreads over many SMs
  CUtensorMap tmWin[3], tmWout[3];
  std::vector<CUtensorMap> tmWconv[3], tmWqkv[3], tmWo[3];
  // float offsets into fconst
  size_t o_bin = 0, o_bout = 0, o_tau = 0;
  std::vector<size_t> o_bconv, o_bqkv, o_bo;
  std::vector<void*> allocs;
  Profiler* prof = nullptr;
  // launch plumbing
  bool pdl = true;                       // programmatic dependent launch between the step's kernels
  int  kv_rs = 0, kv_hs = 0, dh_shift = 0;   // K/V plane layout (see GemmParams)
  int  n_sm = 148;                       // SMs of the device (read at create)
  cudaStream_t cap_stream = nullptr;     // used only to capture graphs at create
  std::map<int, GraphEntry> graphs;      // batch size -> captured chunk step
  uint64_t graph_launches = 0;           // graph launches issued by decode calls
  std::vector<SlotSet> sets;
};

struct FlowState {
  FlowModel* m = nullptr;
  bf16* halo = nullptr;
  bf16* kv = nullptr;
  size_t halo_bytes = 0, kv_bytes = 0;
  long long frames = 0;     // frames appended so far (drives ring head and carried length)
  int       rng_id = 0;     // index of the stream's device random stream
};

namespace {

template <typename T>
cudaError_t dalloc(FlowModel* m, T** p, size_t n, bool zero = true) {
  cudaError_t e = dev_alloc(p, n * sizeof(T));
  if (e != cudaSuccess) return e;
  m->allocs.push_back(*p);
  return zero ? cudaMemset(*p, 0, n * sizeof(T)) : cudaSuccess;
}

// transposes a [K][N] fp32 matrix into bf16 [N][ldk] (K-major rows), zero padded
void pack_wt(std::vector<uint16_t>& dst, size_t off, const float* W, int K, int N, int ldk) {
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) dst[off + (size_t)n * ldk + k] = f32_to_bf16_rne(W[(size_t)k * N + n]);
}

}  // namespace

namespace {
bool build_graph(FlowModel* m, int n, bool tick = false);
}

void flow_model_destroy(FlowModel* m) {
  if (!m) return;
  for (auto& kv : m->graphs) {
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    if (kv.second.graph) cudaGraphDestroy(kv.second.graph);
  }
  if (m->cap_stream) cudaStreamDestroy(m->cap_stream);
  for (void* p : m->allocs) dev_free(p);
  delete m;
}

dc_status flow_model_create(const dc_config& cfg, const float* w, FlowModel** out) {
  FlowModel* m = new (std::nothrow) FlowModel();
  if (!m) return DC_ERR_OOM;
  m->cfg = cfg;
  const int C = m->C = cfg.hidden, mel = m->mel = cfg.mel_dim;
  m->Kin = ((2 * mel + KBLK - 1) / KBLK) * KBLK;
  m->n_pass = cfg.cfg_scale > 0.f ? 2 : 1;
  m->S = cfg.max_batch * m->n_pass;
  m->rows = ((m->S * SLOT_ROWS + TILE_M - 1) / TILE_M) * TILE_M;
  // (a multiple of 8 rows: the attention kernel walks the ring in whole 8-row groups of its swizzled tiles; the extra
  // rows only delay the overwriting of frames that are no longer attended)
  m->Rk = (cfg.kv_cap + cfg.f_chunk + cfg.f_lookahead + 7) & ~7;
  m->P = cfg.f_prompt;
  m->cpa = cfg.n_attn > 0 ? cfg.n_conv / cfg.n_attn : cfg.n_conv;
  const int nL = cfg.n_conv, nA = cfg.n_attn, nS = cfg.n_steps;
  const size_t R = (size_t)GUARD + m->rows;

  // ---- pack weights: every matrix transposed to [N][K] so that both UMMA operands are K-major
  size_t wn = (size_t)C * m->Kin + (size_t)nL * C * 3 * C + (size_t)nA * (3 * (size_t)C * C + (size_t)C * C) + (size_t)mel * C;
  std::vector<uint16_t> hw(wn, 0);
  size_t fn = (size_t)C + (size_t)nL * C + (size_t)nA * 4 * C + mel + (size_t)nS * nL * C;
  std::vector<float> hf(fn, 0.f);
  std::vector<size_t> w_conv(nL), w_qkv(nA), w_o(nA);
  size_t wo = 0, fo = 0, src = 0;
  const size_t w_in = wo;
  pack_wt(hw, wo, w + src, 2 * mel, C, m->Kin);
  wo += (size_t)C * m->Kin;
  src += (size_t)2 * mel * C;
  m->o_bin = fo;
  memcpy(&hf[fo], w + src, C * sizeof(float));
  fo += C;
  src += C;
  std::vector<const float*> Pmat(nL);
  m->o_bconv.resize(nL);
  m->o_bqkv.resize(nA);
  m->o_bo.resize(nA);
  int l = 0;
  const int n_groups = nA > 0 ? nA : 1;
  for (int g = 0; g < n_groups; ++g) {
    for (int j = 0; j < m->cpa; ++j, ++l) {
      w_conv[l] = wo;
      // blob W[tap][c_in][c_out] is one [3C][C] matrix with k = tap*C + c_in
      pack_wt(hw, wo, w + src, 3 * C, C, 3 * C);
      wo += (size_t)C * 3 * C;
      src += (size_t)3 * C * C;
      m->o_bconv[l] = fo;
      memcpy(&hf[fo], w + src, C * sizeof(float));
      fo += C;
      src += C;
      Pmat[l] = w + src;
      src += (size_t)C * C;
    }
    if (nA > 0) {
      w_qkv[g] = wo;
      for (int t = 0; t < 3; ++t) {
        pack_wt(hw, wo, w + src, C, C, C);
        wo += (size_t)C * C;
        src += (size_t)C * C;
      }
      w_o[g] = wo;
      pack_wt(hw, wo, w + src, C, C, C);
      wo += (size_t)C * C;
      src += (size_t)C * C;
      m->o_bqkv[g] = fo;
      memcpy(&hf[fo], w + src, 3 * (size_t)C * sizeof(float));
      fo += 3 * (size_t)C;
      src += 3 * (size_t)C;
      m->o_bo[g] = fo;
      memcpy(&hf[fo], w + src, C * sizeof(float));
      fo += C;
      src += C;
    }
  }
  const size_t w_out = wo;
  pack_wt(hw, wo, w + src, C, mel, C);
  wo += (size_t)mel * C;
  src += (size_t)C * mel;
  m->o_bout = fo;
  memcpy(&hf[fo], w + src, mel * sizeof(float));
  fo += mel;
  src += mel;
  // timestep-bias table tau[s][l][:] = emb(s / n) @ bf16(P_l), evaluated once in double
  m->o_tau = fo;
  {
    const int half = C / 2;
    std::vector<double> emb(C);
    for (int s = 0; s < nS; ++s) {
      const double t = (double)s / nS;
      for (int i = 0; i < half; ++i) {
        const double om = pow(10000.0, -(double)i / half);
        emb[i] = sin(1000.0 * t * om);
        emb[half + i] = cos(1000.0 * t * om);
      }
      for (int ll = 0; ll < nL; ++ll) {
        std::vector<double> acc(C, 0.0);
        for (int k = 0; k < C; ++k) {
          const double e = emb[k];
          const float* prow = Pmat[ll] + (size_t)k * C;
          for (int n = 0; n < C; ++n) acc[n] += e * (double)bf16_to_f32(f32_to_bf16_rne(prow[n]));
        }
        for (int n = 0; n < C; ++n) hf[fo + ((size_t)s * nL + ll) * C + n] = (float)acc[n];
      }
    }
    fo += (size_t)nS * nL * C;
  }

  cudaError_t e = cudaSuccess;
  auto chk = [&](cudaError_t x) { if (e == cudaSuccess) e = x; };
  chk(dalloc(m, &m->wts, wn, false));
  chk(dalloc(m, &m->fconst, fn, false));
  chk(dalloc(m, &m->Xa, R * C));
  chk(dalloc(m, &m->Xb, R * C));
  chk(dalloc(m, &m->ssq, (size_t)(C / 16) * m->rows));
  if (cfg.options & DC_OPT_ROUNDED_NORM) chk(dalloc(m, &m->U, R * C));
  chk(dalloc(m, &m->Q, R * C));
  chk(dalloc(m, &m->O, R * C));
  chk(dalloc(m, &m->Ain, R * m->Kin));
  chk(dalloc(m, &m->xstate, (size_t)m->rows * mel));
  chk(dalloc(m, &m->d_slots, (size_t)m->S));
  chk(dalloc(m, &m->d_err, 1));
  if (e == cudaSuccess) chk(cudaMemcpy(m->wts, hw.data(), wn * sizeof(uint16_t), cudaMemcpyHostToDevice));
  if (e == cudaSuccess) chk(cudaMemcpy(m->fconst, hf.data(), fn * sizeof(float), cudaMemcpyHostToDevice));
  if (e == cudaSuccess)
    chk(cudaFuncSetAttribute(flow_gemm_kernel<false, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM_MAX));
  for (auto fn : {flow_gemm_kernel<false, MODE_INPROJ>, flow_gemm_kernel<false, MODE_CONV>, flow_gemm_kernel<false, MODE_CONV, 64>,
                  flow_gemm_kernel<false, MODE_QKV>, flow_gemm_kernel<false, MODE_OPROJ>,
                  flow_gemm_kernel<false, MODE_OUT>})
    if (e == cudaSuccess) chk(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM_MAX));
  if (e == cudaSuccess)
    chk(cudaFuncSetAttribute(flow_gemm_kernel<true, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM_MAX_PAIR));
  if (e == cudaSuccess && cfg.n_attn > 0)
    chk(cudaFuncSetAttribute(m->P > 0 ? flow_attn_kernel<true, false> : (cfg.head_dim == 64 ? flow_attn_kernel<false, true> : flow_attn_kernel<false, false>),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ATT_SMEM));
  if (e != cudaSuccess) {
    set_error("flow model allocation failed: %s", cudaGetErrorString(e));
    flow_model_destroy(m);
    return e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
  }

  bool ok = true;
  ok &= make_tmap(&m->tmAin, m->Ain, R, m->Kin, A_ROWS);
  ok &= make_tmap(&m->tmXa, m->Xa, R, C, A_ROWS);
  ok &= make_tmap(&m->tmXb, m->Xb, R, C, A_ROWS);
  ok &= make_tmap(&m->tmO, m->O, R, C, A_ROWS);
  if (m->U) ok &= make_tmap(&m->tmU, m->U, R, C, A_ROWS);
  for (int v = 0; v < 3; ++v) {
    const int bn = 64 >> v, bq = 192 >> v, bo = 16;
    ok &= make_tmap(&m->tmWin[v], m->wts + w_in, C, m->Kin, bn);
    ok &= make_tmap(&m->tmWout[v], m->wts + w_out, mel, C, bo);
    m->tmWconv[v].resize(nL);
    m->tmWqkv[v].resize(nA);
    m->tmWo[v].resize(nA);
    for (int i = 0; i < nL; ++i) ok &= make_tmap(&m->tmWconv[v][i], m->wts + w_conv[i], C, 3 * C, bn);
    for (int i = 0; i < nA; ++i) {
      ok &= make_tmap(&m->tmWqkv[v][i], m->wts + w_qkv[i], 3 * C, C, bq);
      ok &= make_tmap(&m->tmWo[v][i], m->wts + w_o[i], C, C, bn);
    }
  }
  if (!ok) {
    set_error("cuTensorMapEncodeTiled failed or is unavailable");
    flow_model_destroy(m);
    return DC_ERR_CUDA;
  }
  m->sets.resize((size_t)(m->S + MAX_SLOTS_PER_SET - 1) / MAX_SLOTS_PER_SET);
  {
    m->pdl = !(cfg.options & DC_OPT_NO_PDL);
    // K/V planes are head-major: the rows one attention CTA streams are contiguous
    m->dh_shift = m->cfg.head_dim == 64 ? 6 : 5;
    m->kv_rs = m->cfg.head_dim;
    m->kv_hs = (m->P + m->Rk) * m->cfg.head_dim;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      m->n_sm = sms;
    if (!(cfg.options & DC_OPT_NO_GRAPH) && cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking) == cudaSuccess) {
      // the two batch sizes that matter are captured now, so that no decode call ever builds a graph:
      // a single stream, and the full batch
      const bool g1 = build_graph(m, m->n_pass);   // a single stream
      const bool gs = m->S > m->n_pass ? build_graph(m, m->S) : g1;
      // ... and one pass of the network over n_steps chunks (wavefront decoding), where the model has room for it
      const int n_wave = cfg.n_steps * m->n_pass;
      if (n_wave <= m->S && n_wave <= MAX_SLOTS_PER_SET) build_graph(m, n_wave, true);
      (void)gs;
    }
    cudaGetLastError();
  }
  *out = m;
  return DC_OK;
}

dc_status flow_state_open(FlowModel* m, FlowState** out) {
  FlowState* s = new (std::nothrow) FlowState();
  if (!s) return DC_ERR_OOM;
  s->m = m;
  s->rng_id = m->streams_opened++;   // (a plain counter: streams of one model are opened from one thread at a time)
  const dc_config& c = m->cfg;
  // one set of carries per pass
  s->halo_bytes = (size_t)m->n_pass * c.n_steps * c.n_conv * HALO * m->C * sizeof(bf16);
  s->kv_bytes = (size_t)m->n_pass * c.n_steps * c.n_attn * 2 * (m->P + m->Rk) * m->C * sizeof(bf16);
  cudaError_t e = dev_alloc(&s->halo, s->halo_bytes);
  if (e == cudaSuccess) e = cudaMemset(s->halo, 0, s->halo_bytes);
  if (e == cudaSuccess && s->kv_bytes) {
    e = dev_alloc(&s->kv, s->kv_bytes);
    if (e == cudaSuccess) e = cudaMemset(s->kv, 0, s->kv_bytes);
  }
  if (e != cudaSuccess) {
    set_error("flow stream allocation failed: %s", cudaGetErrorString(e));
    flow_state_close(s);
    return e == cudaErrorMemoryAllocation ? DC_ERR_OOM : DC_ERR_CUDA;
  }
  *out = s;
  return DC_OK;
}

void flow_state_buffers(const FlowState* s, DevBuf* out, int max_entries, int* n) {
  int k = 0;
  if (k < max_entries) out[k++] = DevBuf{s->halo, s->halo_bytes};
  if (s->kv && k < max_entries) out[k++] = DevBuf{s->kv, s->kv_bytes};
  *n = k;
}

long long flow_state_frames(const FlowState* s) { return s->frames; }
void flow_state_set_frames(FlowState* s, long long frames) { s->frames = frames; }
int flow_state_rng_id(const FlowState* s) { return s->rng_id; }
void flow_state_set_rng_id(FlowState* s, int id) { s->rng_id = id; }

dc_status flow_state_reset(FlowModel*, FlowState* s, cudaStream_t st) {
  // base state: zero left context, empty K/V carry (stale ring rows are never attended)
  if (cudaMemsetAsync(s->halo, 0, s->halo_bytes, st) != cudaSuccess) return DC_ERR_CUDA;
  s->frames = 0;
  return DC_OK;
}

const int* flow_error_word(const FlowModel* m) { return m->d_err; }
uint64_t flow_graph_launches(const FlowModel* m) { return m->graph_launches; }

dc_status flow_selftest_bounded_wait(int max_polls) {
  if (max_polls < 1 || max_polls > 1000000) return DC_ERR_ARG;
  int* d = nullptr;
  if (dev_alloc(&d, sizeof(int)) != cudaSuccess) return DC_ERR_OOM;
  int h = 0;
  cudaError_t e = cudaMemset(d, 0, sizeof(int));
  if (e == cudaSuccess) {
    bounded_wait_selftest_kernel<<<1, 32>>>((uint32_t)max_polls, d);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpy(&h, d, sizeof(int), cudaMemcpyDeviceToHost);
  dev_free(d);
  if (e != cudaSuccess) {
    set_error("bounded-wait self-test failed to run: %s", cudaGetErrorString(e));
    return DC_ERR_CUDA;
  }
  return h == 1 ? DC_ERR_TIMEOUT : (h == 2 ? DC_OK : DC_ERR_CUDA);
}

int flow_take_device_error(FlowModel* m) {
  int v = 0;
  if (cudaMemcpy(&v, m->d_err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  if (v != 0) {
    cudaMemset(m->d_err, 0, sizeof(int));
  }
  return v;
}

void flow_state_close(FlowState* s) {
  if (!s) return;
  if (s->halo) dev_free(s->halo);
  if (s->kv) dev_free(s->kv);
  delete s;
}


void flow_set_profiler(FlowModel* m, Profiler* prof) { m->prof = prof; }



namespace {

// Launch helper: optional programmatic-dependent-launch attribute, optional event bracketing.
struct LaunchCtx {
  cudaStream_t st;
  bool         pdl;
  Profiler*    prof;
  int          launches = 0;
  cudaError_t  err = cudaSuccess;
  int          cluster_x = 1;   // > 1: the next launch is a cluster launch of that many CTAs along x
};

template <typename... KArgs, typename... Args>
void launch(LaunchCtx& lc, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, bool pdl_ok, int cls, Args&&... args) {
  ProfScope ps(lc.prof, cls, lc.st);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = lc.st;
  cudaLaunchAttribute attr[2];
  cfg.attrs = attr;
  if (lc.pdl && pdl_ok) {
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    ++cfg.numAttrs;
  }
  if (lc.cluster_x > 1) {   // set by the caller for this one launch
    attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
    attr[cfg.numAttrs].val.clusterDim.x = (unsigned)lc.cluster_x;
    attr[cfg.numAttrs].val.clusterDim.y = 1;
    attr[cfg.numAttrs].val.clusterDim.z = 1;
    ++cfg.numAttrs;
    lc.cluster_x = 1;
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
  if (e != cudaSuccess && lc.err == cudaSuccess) lc.err = e;
  ++lc.launches;
}

// Issues every kernel of one chunk step for n slots (the slot table is uploaded by the first
// kernel(s) from `sets`).
// tick = false: the n slots' chunks, all Euler steps.  tick = true: ONE pass of the network, every slot at the Euler step
// that its slot-table entry encodes (wavefront decoding: the slots are consecutive chunks of one stream).
void enqueue_chunk(FlowModel* m, int n, const SlotSet* sets, int n_sets, LaunchCtx& lc, bool tick = false) {
  const dc_config& c = m->cfg;
  const int C = m->C, mel = m->mel;
  for (int i = 0; i < n_sets; ++i)   // not a programmatic launch: it overwrites the table the previous chunk still reads
    launch(lc, set_slots_kernel, dim3(1), dim3(MAX_SLOTS_PER_SET), 0, false, 4, sets[i], m->d_slots);
  launch(lc, flow_prep_kernel, dim3(n), dim3(128), 0, true, 4, (const SlotInfo*)m->d_slots, mel, m->xstate, m->Ain, m->Kin,
         (uint32_t)c.noise_seed_lo, (uint32_t)c.noise_seed_hi);

  const int m_tiles = (n * SLOT_ROWS + TILE_M - 1) / TILE_M;
  // N-tile variant: the narrowest whose C-wide GEMMs still fit ONE wave (a GEMM CTA has an SM to itself);
  // a second, part-filled wave costs more than wider tiles do (measured with 5 and 10 row tiles: 160 CTAs
  // of 16 columns 0.26 ms per pass, 80 CTAs of 32 columns 0.20 ms)
  int v = 2;
  while (v > 0 && m_tiles * (C / (64 >> v)) > m->n_sm) --v;
  // the output projection always uses 16-column tiles: mel/16 CTAs per row tile instead of one, and a
  // single Euler-state round trip per epilogue thread
  const int bn = 64 >> v, bq = 192 >> v, bo = 16;
  // CTA pairs (DC_OPT_CTA_PAIRS): full batches only (the widest tiles, an even number of row tiles), and only the
  // GEMMs whose weight tile is a large part of a stage; tBh is the same weight matrix with boxes of BN / 2 rows
  const bool pairs_ok = v == 0 && m_tiles % 2 == 0 && (c.options & DC_OPT_CTA_PAIRS);
  auto gemm = [&](const CUtensorMap& tA, const CUtensorMap& tB, GemmParams& p, int N, const CUtensorMap* tBh = nullptr) {
    p.n_slots = n;
    p.slots = m->d_slots;
    p.ld = C;
    p.C = C;
    p.Rk = m->Rk;
    p.P = m->P;
    p.err = m->d_err;
    p.empty = (c.options & DC_OPT_EMPTY_KERNELS) ? 1 : 0;
    const int stage_bytes = A_BYTES + p.taps * ((p.BN * 128 + 1023) & ~1023);
    // the issuer count fixes the summation order, so it depends on the GEMM's role only, never on the tile
    // width chosen for the batch size (batched and single-stream results must agree bit for bit);
    // the QKV and output projections keep one issuer (their wide tiles would not fit two accumulators)
    p.n_issuers = (p.mode != MODE_QKV && p.mode != MODE_OUT && p.n_kblocks >= 2) ? 2 : 1;
    // Stage count.  With two issuers the count must be EVEN: issuer i takes
    // the reduction blocks kb = i (mod 2), and only with an even ring does every stage always belong
    // to the same issuer - a parity wait cannot tell "my block has landed" from "the other issuer's
    // earlier block has landed" on a stage that both use.
    if (p.n_issuers == 2) {
      p.n_stages = (p.n_kblocks >= 4 && (4 * stage_bytes <= 104 * 1024 || stage_bytes > 32 * 1024)) ? 4 : 2;
    } else {
      p.n_stages = std::max(1, std::min(std::min(MAX_STAGES, GEMM_TILE_SMEM / stage_bytes), p.n_kblocks));
      // the wide QKV tiles fill the GPU with one CTA per SM anyway: a deeper ring hides the load latency
      if (p.mode == MODE_QKV && stage_bytes > 32 * 1024 && p.n_kblocks >= 4) p.n_stages = 4;
    }
    if (pairs_ok && tBh != nullptr) {
      const int pair_stage = A_BYTES + p.taps * (p.BN * 64);
      int ns = p.n_kblocks < MAX_STAGES ? p.n_kblocks : MAX_STAGES;
      while (ns > 1 && GEMM_SMEM_EXTRA + (size_t)ns * pair_stage > GEMM_SMEM_MAX_PAIR) --ns;
      if (p.n_issuers == 2) ns &= ~1;
      // the conv epilogue exchanges shifted rows through 64 KB of the (by then idle) ring
      if (ns >= 2 && (size_t)ns * pair_stage >= 64 * 1024) {
        p.n_stages = ns;
        lc.cluster_x = 2;
        launch(lc, flow_gemm_kernel<true, -1>, dim3(m_tiles, N / p.BN), dim3(GEMM_THREADS), GEMM_SMEM_EXTRA + (size_t)ns * pair_stage, true,
               7, tA, *tBh, p);
        return;
      }
    }
    const size_t smem = GEMM_SMEM_EXTRA + (size_t)p.n_stages * stage_bytes;
    // One instantiation per role for batches of eight row tiles or more: the other roles' epilogues and the slot
    // fields only they read then cost neither registers nor instructions (32 streams: 2.01 -> 1.94 ms per step).
    // Small batches keep the one generic kernel for every role: their launches are so short that five alternating
    // kernel images cost more in instruction-cache misses than the leaner code saves (1 stream: 1.37 -> 1.46 ms
    // with the specialised forms; the two break even between 4 and 8 row tiles).
    const dim3 grid(m_tiles, N / p.BN);
    const int cls = p.mode == MODE_CONV ? 0 : 1;
    if (m_tiles < SPECIALISE_FROM_TILES) launch(lc, flow_gemm_kernel<false, -1>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    // (a conv block's widest tile, that of a full batch, also has its width fixed at compile time - the epilogue's chunk
    // loop unrolls away: 1.94 -> 1.91 ms per step; the same for the other roles, or a second conv image per kind of
    // tail - carried rows / row statistics - measured nothing or cost what another kernel image costs)
    else if (p.mode == MODE_CONV && p.n_issuers == 2 && p.BN == 64)
      launch(lc, flow_gemm_kernel<false, MODE_CONV, 64>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else if (p.mode == MODE_CONV && p.n_issuers == 2) launch(lc, flow_gemm_kernel<false, MODE_CONV>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else if (p.mode == MODE_QKV) launch(lc, flow_gemm_kernel<false, MODE_QKV>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else if (p.mode == MODE_OPROJ) launch(lc, flow_gemm_kernel<false, MODE_OPROJ>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else if (p.mode == MODE_INPROJ) launch(lc, flow_gemm_kernel<false, MODE_INPROJ>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else if (p.mode == MODE_OUT) launch(lc, flow_gemm_kernel<false, MODE_OUT>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
    else launch(lc, flow_gemm_kernel<false, -1>, grid, dim3(GEMM_THREADS), smem, true, cls, tA, tB, p);
  };
  // the GEMM whose output feeds an RMS norm leaves the row statistics; the GEMM after the norm applies them
  auto feeds_norm = [&](GemmParams& p) { p.ssq_out = m->ssq; p.ssq_ld = m->rows; };
  auto normalised = [&](GemmParams& p) {
    p.ssq_in = m->ssq; p.ssq_ld = m->rows; p.inv_C = 1.0f / (float)C; p.eps = c.rms_eps;
  };
  // DC_OPT_ROUNDED_NORM: a kernel of its own writes u = bf16(x / rms) and the projection reads u unscaled
  const bool rounded_norm = m->U != nullptr;
  auto rmsnorm = [&](const bf16* x) {
    const int warps = n * SLOT_ROWS;
    launch(lc, flow_rmsnorm_kernel, dim3((warps * 32 + 255) / 256), dim3(256), 0, true, 3, (const SlotInfo*)m->d_slots, n, x, m->U, C,
           (const float*)m->ssq, (long long)m->rows, 1.0f / (float)C, c.rms_eps);
  };
  auto attention = [&](int step, int layer) {
    AttnParams p{};
    p.slots = m->d_slots; p.q = m->Q; p.o = m->O; p.ld = C; p.dh = c.head_dim;
    p.kv_off = ((long long)step * c.n_attn + layer) * 2 * (m->P + m->Rk) * C;
    p.Rk = m->Rk; p.C = C; p.P = m->P;
    p.kv_rs = m->kv_rs; p.kv_hs = m->kv_hs;
    p.scale_log2e = (float)(1.4426950408889634 / sqrt((double)c.head_dim));
    p.err = m->d_err;
    p.empty = (c.options & DC_OPT_EMPTY_KERNELS) ? 1 : 0;
    launch(lc, m->P > 0 ? flow_attn_kernel<true, false> : (c.head_dim == 64 ? flow_attn_kernel<false, true> : flow_attn_kernel<false, false>),
           dim3(n, c.n_heads), dim3(ATT_THREADS), ATT_SMEM, true, 2, p);
  };
  const float* fc = m->fconst;
  const long long halo_stride = (long long)HALO * C;

  for (int s = 0; s < (tick ? 1 : c.n_steps); ++s) {
    bf16* X = m->Xa;                 // current residual stream
    bf16* Y = m->Xb;
    const CUtensorMap* tX = &m->tmXa;
    const CUtensorMap* tY = &m->tmXb;
    auto swap = [&]() { std::swap(X, Y); std::swap(tX, tY); };
    {
      GemmParams p{};
      p.mode = MODE_INPROJ; p.BN = bn; p.n_kblocks = m->Kin / KBLK; p.taps = 1;
      p.bias = fc + m->o_bin; p.out = X;
      p.halo_off = ((long long)s * c.n_conv + 0) * halo_stride;
      if (m->cpa == 0) feeds_norm(p);
      gemm(m->tmAin, m->tmWin[v], p, C);
    }
    int l = 0;
    const int n_groups = c.n_attn > 0 ? c.n_attn : 1;
    for (int g = 0; g < n_groups; ++g) {
      for (int j = 0; j < m->cpa; ++j, ++l) {
        const int d = c.dilations[l];
        GemmParams p{};
        p.mode = MODE_CONV; p.BN = bn; p.n_kblocks = C / KBLK; p.taps = 3;
        p.shift[0] = 2 * d; p.shift[1] = d; p.shift[2] = 0;
        p.bias = fc + m->o_bconv[l]; p.tau = fc + m->o_tau + ((size_t)s * c.n_conv + l) * C;
        p.resid = X; p.out = Y;
        const bool next_is_conv = (j + 1 < m->cpa);
        p.halo_off = next_is_conv ? ((long long)s * c.n_conv + l + 1) * halo_stride : -1;
        if (!next_is_conv) feeds_norm(p);   // the group's attention norm, or the final norm of a conv-only stack
        if (!(c.options & DC_OPT_SKIP_CONV_GEMM)) gemm(*tX, m->tmWconv[v][l], p, C, &m->tmWconv[1][l]);   // (measurement only: the step without this class)
        swap();
      }
      if (c.n_attn > 0) {
        {
          GemmParams p{};
          p.mode = MODE_QKV; p.BN = bq; p.n_kblocks = C / KBLK; p.taps = 1;
          p.bias = fc + m->o_bqkv[g]; p.q_out = m->Q; p.halo_off = -1;
          p.kv_off = ((long long)s * c.n_attn + g) * 2 * (m->P + m->Rk) * C;
          p.kv_rs = m->kv_rs; p.kv_hs = m->kv_hs; p.dh_shift = m->dh_shift;
          if (rounded_norm) {
            rmsnorm(X);
            gemm(m->tmU, m->tmWqkv[v][g], p, 3 * C, &m->tmWqkv[1][g]);
          } else {
            normalised(p);
            gemm(*tX, m->tmWqkv[v][g], p, 3 * C, &m->tmWqkv[1][g]);
          }
        }
        if (!(c.options & DC_OPT_SKIP_ATTENTION)) attention(s, g);   // (measurement only: the step without this class)
        {
          GemmParams p{};
          p.mode = MODE_OPROJ; p.BN = bn; p.n_kblocks = C / KBLK; p.taps = 1;
          p.bias = fc + m->o_bo[g]; p.resid = X; p.out = Y;
          p.halo_off = (l < c.n_conv) ? ((long long)s * c.n_conv + l) * halo_stride : -1;
          if (g == n_groups - 1 || m->cpa == 0) feeds_norm(p);   // final norm, or the next group's norm
          gemm(m->tmO, m->tmWo[v][g], p, C);
          swap();
        }
      }
    }
    {
      GemmParams p{};
      p.mode = MODE_OUT; p.BN = bo; p.n_kblocks = C / KBLK; p.taps = 1;
      p.bias = fc + m->o_bout; p.halo_off = -1;
      p.xstate = m->xstate; p.ain = m->Ain; p.ld_ain = m->Kin; p.inv_n = 1.0f / c.n_steps;
      p.last_step = (!tick && s == c.n_steps - 1); p.mel = mel; p.cfg_w = c.cfg_scale;
      if (rounded_norm) {
        rmsnorm(X);
        gemm(m->tmU, m->tmWout[v], p, mel);
      } else {
        normalised(p);
        gemm(*tX, m->tmWout[v], p, mel);
      }
    }
  }
}

// One captured graph per batch size: the whole chunk step becomes a single graph launch; only the
// slot-table node's by-value argument changes from call to call.
// Graphs are keyed by the slot count; tick graphs (one pass of the network, wavefront decoding) by its negative.
bool build_graph(FlowModel* m, int n, bool tick) {
  if (n > MAX_SLOTS_PER_SET || m->cap_stream == nullptr) return false;
  for (int use_pdl = m->pdl ? 1 : 0; use_pdl >= 0; --use_pdl) {
    SlotSet dummy{};
    dummy.first = 0;
    dummy.count = 0;
    cudaGraph_t graph = nullptr;
    if (cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    LaunchCtx lc{m->cap_stream, use_pdl != 0, nullptr};
    enqueue_chunk(m, n, &dummy, 1, lc, tick);
    cudaError_t e = cudaStreamEndCapture(m->cap_stream, &graph);
    if (e != cudaSuccess || lc.err != cudaSuccess || graph == nullptr) {
      cudaGetLastError();
      if (graph) cudaGraphDestroy(graph);
      continue;
    }
    GraphEntry ge{};
    size_t n_nodes = 0;
    cudaGraphGetNodes(graph, nullptr, &n_nodes);
    std::vector<cudaGraphNode_t> nodes(n_nodes);
    cudaGraphGetNodes(graph, nodes.data(), &n_nodes);
    for (cudaGraphNode_t nd : nodes) {
      cudaGraphNodeType ty;
      if (cudaGraphNodeGetType(nd, &ty) != cudaSuccess || ty != cudaGraphNodeTypeKernel) continue;
      cudaKernelNodeParams kp{};
      if (cudaGraphKernelNodeGetParams(nd, &kp) == cudaSuccess && kp.func == (void*)set_slots_kernel) ge.set_node = nd;
    }
    e = cudaGraphInstantiate(&ge.exec, graph, 0);
    if (e != cudaSuccess || ge.set_node == nullptr) {
      cudaGetLastError();
      if (ge.exec) cudaGraphExecDestroy(ge.exec);
      cudaGraphDestroy(graph);
      continue;
    }
    ge.graph = graph;
    ge.launches = lc.launches;
    ge.pdl = use_pdl != 0;
    m->graphs[tick ? -n : n] = ge;
    return true;
  }
  return false;
}

}  // namespace

dc_status flow_decode(FlowModel* m, int n, FlowState* const* states, const float* const* feats, const int* T,
                      float* const* outp, cudaStream_t st, int* launches) {
  const dc_config& c = m->cfg;
  // ---- per-call slot table (passed by value through a kernel, so nothing is staged or allocated);
  // with guidance a stream takes two adjacent slots, one per pass
  const int n_streams = n;
  const int np = m->n_pass;
  n = n_streams * np;                         // slots from here on
  const int n_sets = (n + MAX_SLOTS_PER_SET - 1) / MAX_SLOTS_PER_SET;
  std::vector<SlotSet>& sets = m->sets;   // sized at create
  for (int k = 0; k < n_sets; ++k) {
    SlotSet& set = sets[(size_t)k];
    set.first = k * MAX_SLOTS_PER_SET;
    set.count = n - set.first < MAX_SLOTS_PER_SET ? n - set.first : MAX_SLOTS_PER_SET;
    for (int i = 0; i < set.count; ++i) {
      const int stream = (set.first + i) / np, pass = (set.first + i) % np;
      FlowState* s = states[stream];
      SlotInfo& si = set.s[i];
      si.T = T[stream];
      const long long hist = s->frames > m->P ? s->frames - m->P : 0;   // history frames so far (after the prompt)
      si.n_prompt0 = (int)(s->frames < m->P ? s->frames : m->P);
      si.kv_head = (int)(hist % m->Rk);
      si.kv_len = (int)(hist < c.kv_cap ? hist : c.kv_cap);
      si.Tc = si.T < c.f_chunk ? si.T : c.f_chunk;
      si.frame0 = s->frames;
      si.rng_id = s->rng_id;
      si.tau_off = 0;
      si.flags = SLOT_FIRST;
      si.pad = 0;
      si.pass = pass;
      si.feats = feats[stream];
      si.out = pass == 0 ? outp[stream] : nullptr;
      si.halo = s->halo + (size_t)pass * (s->halo_bytes / sizeof(bf16) / np);
      si.kv = s->kv ? s->kv + (size_t)pass * (s->kv_bytes / sizeof(bf16) / np) : nullptr;
    }
  }
  const bool profiling = m->prof != nullptr && m->prof->on;
  auto it = m->graphs.find(n);
  // a batch size met for the first time captures its chunk step now (one graph per size, kept for the model's
  // lifetime: the finite catalog of launch shapes), so that every admitted call is one graph launch
  if (it == m->graphs.end() && !profiling && build_graph(m, n)) it = m->graphs.find(n);
  if (!profiling && it != m->graphs.end()) {
    // one launch for the whole chunk step
    GraphEntry& ge = it->second;
    void* args[2] = {&sets[0], &m->d_slots};
    cudaKernelNodeParams kp{};
    kp.func = (void*)set_slots_kernel;
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(MAX_SLOTS_PER_SET);
    kp.sharedMemBytes = 0;
    kp.kernelParams = args;
    kp.extra = nullptr;
    cudaError_t e = cudaGraphExecKernelNodeSetParams(ge.exec, ge.set_node, &kp);
    if (e == cudaSuccess) e = cudaGraphLaunch(ge.exec, st);
    if (e != cudaSuccess) {
      set_error("flow decode graph launch failed: %s", cudaGetErrorString(e));
      return DC_ERR_CUDA;
    }
    *launches += ge.launches;
    ++m->graph_launches;
  } else {
    LaunchCtx lc{st, m->pdl && !profiling, m->prof};
    enqueue_chunk(m, n, sets.data(), n_sets, lc);
    *launches += lc.launches;
    if (lc.err != cudaSuccess || cudaGetLastError() != cudaSuccess) {
      set_error("flow decode launch failed: %s", cudaGetErrorString(lc.err));
      return DC_ERR_CUDA;
    }
  }
  for (int i = 0; i < n_streams; ++i) states[i]->frames += T[i] < c.f_chunk ? T[i] : c.f_chunk;
  return DC_OK;
}

// Wavefront decoding of streams whose input is all there: chunk j of a stream runs its Euler step s in tick
// j + s, so a tick is one pass of the network over n_steps consecutive chunks of every stream, each at its own
// step.  Chunk j at step s needs the step-s carries that chunk j-1 left one tick earlier, and chunks that share a
// tick use the carries of different steps, so every tick is free of read/write conflicts.  A chunk keeps slot
// (j mod n_steps) of its stream's slots for its n_steps ticks (its Euler state lives there); slots of chunks not
// yet started or already finished are holes (T = 0).  The arithmetic of a slot never depends on what the other
// slots hold, so the result equals chunk-by-chunk decoding bit for bit.
dc_status flow_decode_wave(FlowModel* m, int n_streams, FlowState* const* states, const float* const* feats, int in_dim,
                           const long long* n_frames, float* const* outs, cudaStream_t st, int* launches,
                           void (*on_chunk)(void*, int, long long), void* hook_ctx) {
  const dc_config& c = m->cfg;
  const int np = m->n_pass, K = c.n_steps;
  const int n = n_streams * K * np;                       // slots of a tick
  if (n_streams < 1 || n > m->S || n > MAX_SLOTS_PER_SET) {
    set_error("wavefront decoding keeps n_steps = %d chunks per stream in flight: %d streams need max_batch >= %d (and at most %d slots)",
              K, n_streams, n_streams * K, MAX_SLOTS_PER_SET);
    return DC_ERR_ARG;
  }
  long long max_chunks = 0;
  for (int i = 0; i < n_streams; ++i) {
    const long long nc = (n_frames[i] + c.f_chunk - 1) / c.f_chunk;
    if (nc > max_chunks) max_chunks = nc;
  }
  const bool profiling = m->prof != nullptr && m->prof->on;
  auto it = m->graphs.find(-n);   // one stream: captured at create; other stream counts: at their first call
  if (it == m->graphs.end() && !profiling && build_graph(m, n, true)) it = m->graphs.find(-n);
  const size_t halo_step = (size_t)c.n_conv * HALO * m->C, kv_step = (size_t)c.n_attn * 2 * (m->P + m->Rk) * m->C;
  SlotSet& set = m->sets[0];
  for (long long t = 0; t < max_chunks + K - 1; ++t) {
    set.first = 0;
    set.count = n;
    for (int i = 0; i < n; ++i) {
      SlotInfo& si = set.s[i];
      si = SlotInfo{};
      const int stream = i / (K * np), ring = (i / np) % K, pass = i % np;
      const FlowState* s = states[stream];
      const long long n_chunks = (n_frames[stream] + c.f_chunk - 1) / c.f_chunk;
      // the chunk that owns ring slot `ring` in tick t: the largest j <= t with j = ring (mod K)
      const long long j = t - (((t - ring) % K) + K) % K;
      const long long step = t - j;
      if (j < 0 || j >= n_chunks || step >= K) continue;                  // hole
      const long long f0 = j * c.f_chunk, left = n_frames[stream] - f0;
      const long long frames = s->frames + f0;
      si.T = (int)(left < c.f_chunk + c.f_lookahead ? left : c.f_chunk + c.f_lookahead);
      si.Tc = si.T < c.f_chunk ? si.T : c.f_chunk;
      const long long hist = frames > m->P ? frames - m->P : 0;
      si.n_prompt0 = (int)(frames < m->P ? frames : m->P);
      si.kv_head = (int)(hist % m->Rk);
      si.kv_len = (int)(hist < c.kv_cap ? hist : c.kv_cap);
      si.frame0 = frames;
      si.rng_id = s->rng_id;
      si.tau_off = (int)(step * c.n_conv * m->C);
      si.flags = (step == 0 ? SLOT_FIRST : 0) | (step == K - 1 ? SLOT_LAST : 0);
      si.pass = pass;
      si.feats = feats[stream] + f0 * in_dim;
      si.out = pass == 0 ? outs[stream] + f0 * m->mel : nullptr;
      si.halo = s->halo + (size_t)pass * (s->halo_bytes / sizeof(bf16) / np) + (size_t)step * halo_step;
      si.kv = s->kv ? s->kv + (size_t)pass * (s->kv_bytes / sizeof(bf16) / np) + (size_t)step * kv_step : nullptr;
    }
    if (!profiling && it != m->graphs.end()) {
      GraphEntry& ge = it->second;
      void* args[2] = {&set, &m->d_slots};
      cudaKernelNodeParams kp{};
      kp.func = (void*)set_slots_kernel;
      kp.gridDim = dim3(1);
      kp.blockDim = dim3(MAX_SLOTS_PER_SET);
      kp.kernelParams = args;
      cudaError_t e = cudaGraphExecKernelNodeSetParams(ge.exec, ge.set_node, &kp);
      if (e == cudaSuccess) e = cudaGraphLaunch(ge.exec, st);
      if (e != cudaSuccess) {
        set_error("wavefront graph launch failed: %s", cudaGetErrorString(e));
        return DC_ERR_CUDA;
      }
      *launches += ge.launches;
      ++m->graph_launches;
    } else {
      LaunchCtx lc{st, m->pdl && !profiling, m->prof};
      enqueue_chunk(m, n, &set, 1, lc, true);
      *launches += lc.launches;
      if (lc.err != cudaSuccess || cudaGetLastError() != cudaSuccess) {
        set_error("wavefront launch failed: %s", cudaGetErrorString(lc.err));
        return DC_ERR_CUDA;
      }
    }
    if (on_chunk && t >= K - 1)   // the last Euler step of every stream's chunk t - (K - 1) is now enqueued
      for (int i = 0; i < n_streams; ++i)
        if (t - (K - 1) < (n_frames[i] + c.f_chunk - 1) / c.f_chunk) on_chunk(hook_ctx, i, t - (K - 1));
  }
  for (int i = 0; i < n_streams; ++i) states[i]->frames += n_frames[i];
  return DC_OK;
}


}  // namespace dc
