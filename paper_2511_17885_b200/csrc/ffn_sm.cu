// Expert FFNs on the tcgen05 tensor cores, small-M form: the token rows are the MMA's N dimension.
//
// Section 3.1 makes the rows per expert small on purpose: a vision token activates K_v < K experts, so
// at batch 1 an expert sees a few dozen to ~120 rows (and a decode step a handful).  With the rows as
// the MMA's M dimension (ffn_tc.cu) every k-step pays a full 128-row instruction and loads a 128-row
// activation box whatever the row count.  Here the roles are swapped:
//   D[128 output features, N token rows] (+)= W[128 features, 64] * X[N rows, 64]^T,   N = 16, 32, ... 128
// so that the tensor work of a tile and the activation box both shrink with the expert's rows, in steps
// of 16 and 32 rows.  Everything else is the persistent kernel of ffn_tc.cu: the same tile list and
// interleaved order, a warp that schedules tiles, one that feeds a 4-stage TMA ring, one thread that issues
// the MMAs into two tensor-memory accumulator stages, four epilogue warps.
//   GEMM-1: a tile is (M-tile of one expert) x (128 intermediate features); two MMAs per k-step (gate
//           rows, up rows) share the activation operand; accumulators D_gate, D_up hold feature f in
//           TMEM lane f and token t in column t, so one thread owns gate and up of (f, t): SwiGLU in
//           registers, then act[row0 + t][f] with the warp's 32 lanes writing 32 neighbouring features.
//   GEMM-2: a tile is (M-tile) x (256 hidden features) as two MMAs (features 0-127, 128-255); the
//           epilogue scales by the token's gate and adds the warp's 32 neighbouring features of one
//           token to the fp32 accumulator with one 128-byte reduction (or stores them, fixed-order mode).
// The transposed accumulator needs no shared-memory staging: for a fixed token the lanes of a warp already
// hold consecutive output features.
// When it runs: bf16 layers below 256 tokens (decode-sized batches; from there on the rows-as-M form with
// the in-GEMM row gather measured faster) and every layer with FP8 weights.
// FP8 weight stream (WQ = 1): the expert matrices arrive as FP8 E4M3 bytes with one power-of-two scale per
// 128 x 128 block.  TMA brings the bytes (half the HBM traffic of bf16) into a ring of raw stages; eight more
// warps expand every weight box to bf16 in the 128-byte-swizzled layout the MMA reads (exactly: an E4M3 value
// has 4 significant bits and the scale is a power of two) into a second, two-deep ring; the activations stay
// bf16 and go from the raw stage straight to the MMA.  The contraction, the accumulators and the epilogues are
// those of the bf16 stream.
// Every wait is bounded; on expiry the CTA records FMMOE_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"
#include "ffn_common.cuh"

namespace fmmoe {

constexpr int S_BK = 64;                              // one 128-byte swizzle atom of bf16
constexpr int S_STAGES = 4;
constexpr int S_W_BYTES = 128 * S_BK * 2;             // one 128-feature weight box as bf16: 16 KB
constexpr int S_WQ_BYTES = 128 * S_BK;                // the same box as FP8 bytes: 8 KB
constexpr int S_X_BYTES = 128 * S_BK * 2;             // room for up to 128 token rows: 16 KB
constexpr int S_THREADS = 224;                        // producer warp, issuer warp, four epilogue warps, tile-scheduler warp
constexpr int S_CONVERTERS = 256;                     // FP8 stream: eight more warps that expand the weight boxes
constexpr int S_CVT_PIECES = 512 / S_CONVERTERS;      // 16-byte pieces of a weight box per converter thread
constexpr int S_CVT_STAGES = 2;
constexpr int S_TMEM_COLS = 512;                      // 2 accumulator stages x (2 x 128 columns)
// bf16 stream: a stage is [W0 16K][W1 16K][X 16K].  FP8 stream: a raw stage is [W0 8K][W1 8K][X 16K] and the
// expanded weights live in S_CVT_STAGES buffers of [W0 16K][W1 16K].
template <int WQ> struct SmLayout {
  static constexpr int W_RAW = WQ ? S_WQ_BYTES : S_W_BYTES;
  static constexpr int X_OFF = 2 * W_RAW;
  static constexpr int STAGE_BYTES = X_OFF + S_X_BYTES;
  static constexpr int CVT_OFF = S_STAGES * STAGE_BYTES;
  static constexpr int CVT_BYTES = WQ ? S_CVT_STAGES * 2 * S_W_BYTES : 0;
  static constexpr int BAR_OFF = CVT_OFF + CVT_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 1024 /*align*/ + 512 /*barriers, tile ring*/;
  static constexpr int THREADS = WQ ? S_THREADS + S_CONVERTERS : S_THREADS;
};

// Two E4M3 bytes (bytes 2*sel and 2*sel+1 of w) -> two bf16 in one word, times `mul` (a power of two in both
// halves).  An E4M3 byte s.eeee.mmm placed as s.0000eeee.mmm0000 is the bf16 number 2^(e-127) (1 + m/8), or the
// bf16 subnormal 2^-126 (m/8) for e = 0: in both cases the E4M3 value times 2^-120, so one exact bf16 multiply
// by 2^(120 + scale exponent) finishes the conversion.
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t w, int sel, __nv_bfloat162 mul) {
  const uint32_t y = __byte_perm(w, 0u, sel ? 0x3424u : 0x1404u);     // [b_lo << 8 | b_hi << 24]
  const uint32_t bits = (y & 0x80008000u) | ((y >> 4) & 0x07f007f0u);
  const __nv_bfloat162 v = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&bits), mul);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ void red_add_f32(float* addr, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(v) : "memory");
}

// Token rows of a tile as the MMA sees them: a multiple of 16 (the instruction's N granularity for M = 128).
__device__ __forceinline__ int n_pad_of(int rows) { return rows <= 16 ? 16 : (rows + 15) & ~15; }

// MODE 0: GEMM-1 + SwiGLU.  MODE 1: GEMM-2 + combine.
template <int MODE, int WQ>
__global__ void __launch_bounds__(SmLayout<WQ>::THREADS, 1)
ffn_sm_kernel(const __grid_constant__ CUtensorMap tmX32, const __grid_constant__ CUtensorMap tmX64,
              const __grid_constant__ CUtensorMap tmX96, const __grid_constant__ CUtensorMap tmX128,
              const __grid_constant__ CUtensorMap tmXs,
              const __grid_constant__ CUtensorMap tmW0_r, const __grid_constant__ CUtensorMap tmW1_r,
              const __grid_constant__ CUtensorMap tmW0_s, const __grid_constant__ CUtensorMap tmW1_s,
              const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + ((1024 - (raw & 1023)) & 1023);   // 1024-byte aligned tiles (128B swizzle)
  using L = SmLayout<WQ>;
  constexpr int S_STAGE_BYTES = L::STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::BAR_OFF);
  uint64_t* full_bar = bars;                   // [S_STAGES]
  uint64_t* empty_bar = bars + S_STAGES;       // [S_STAGES]
  uint64_t* tfull_bar = bars + 2 * S_STAGES;   // [2]
  uint64_t* tempty_bar = tfull_bar + 2;        // [2]
  uint64_t* sfull_bar = tempty_bar + 2;        // [G_SCHED]
  uint64_t* sempty_bar = sfull_bar + G_SCHED;  // [G_SCHED]
  uint64_t* cfull_bar = sempty_bar + G_SCHED;  // [S_CVT_STAGES]  FP8 stream: expanded weights ready
  uint64_t* cempty_bar = cfull_bar + S_CVT_STAGES;   // [S_CVT_STAGES]
  volatile int* ring = reinterpret_cast<volatile int*>(cempty_bar + S_CVT_STAGES);   // [G_SCHED][G_SLOT_INTS]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ring) + G_SCHED * G_SLOT_INTS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* prod_half = abort_flag + 1;    // tiles the producer has taken half-way (paces the tile scheduler)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t budget = p.wait_budget_ns;
  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    // a raw stage is free again once the MMAs have read its activations and (FP8 stream) every converter
    // warp has read its weight bytes (one arrival per warp: hundreds of per-thread arrivals on one barrier
    // would cost more than the conversion itself)
    for (int i = 0; i < S_STAGES; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], WQ ? 1 + S_CONVERTERS / 32 : 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull_bar[i], 1); mbar_init(&tempty_bar[i], 128); }
    // readers of a tile id: producer + issuer + 4 epilogue warps (+ the converter warps)
    for (int i = 0; i < G_SCHED; ++i) { mbar_init(&sfull_bar[i], 1); mbar_init(&sempty_bar[i], WQ ? 6 + S_CONVERTERS / 32 : 6); }
    for (int i = 0; i < S_CVT_STAGES; ++i) { mbar_init(&cfull_bar[i], S_CONVERTERS / 32); mbar_init(&cempty_bar[i], 1); }
    *abort_flag = 0;
    *prod_half = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, S_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // barriers, tensor memory and descriptors are set up; everything below reads what earlier
  // kernels of the stream wrote
  pdl_wait();
  const int n_mt_r = p.n_mtiles ? min(max(*p.n_mtiles, 0), p.max_mtiles) : 0;
  const int total_tiles = n_mt_r * p.seg[0].n_nblocks + p.shared_mtiles * p.seg[1].n_nblocks;

  if (warp == 0) {
    // ------------------------------------------------------------ scheduler + TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmX32); tma_prefetch_desc(&tmX64); tma_prefetch_desc(&tmX96); tma_prefetch_desc(&tmX128);
      tma_prefetch_desc(&tmW0_r); tma_prefetch_desc(&tmW1_r);
      if (p.shared_mtiles) { tma_prefetch_desc(&tmXs); tma_prefetch_desc(&tmW0_s); tma_prefetch_desc(&tmW1_s); }
      const uint64_t pol_stream = l2_policy_evict_first();
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      int issued = 0;        // k-blocks handed to the TMA engine so far
      bool stop = false;
      for (uint32_t it = 0; ok && !stop; ++it) {
        // the tile comes decoded from the scheduler warp: the producer touches no global memory but the TMA maps
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag, budget)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const Segment& sg = p.seg[ti.seg];
        // activation box: the smallest of 32 / 64 / 96 / 128 rows that covers the tile's (padded) rows
        const int npad = n_pad_of(ti.rows);
        const int bi = ti.seg ? 3 : (npad + 31) / 32 - 1;
        const CUtensorMap* mX = ti.seg ? &tmXs : (bi == 0 ? &tmX32 : bi == 1 ? &tmX64 : bi == 2 ? &tmX96 : &tmX128);
        const uint32_t x_bytes = (uint32_t)(bi + 1) * 32u * 128u;
        const CUtensorMap* mW0 = ti.seg ? &tmW0_s : &tmW0_r;
        const CUtensorMap* mW1 = ti.seg ? &tmW1_s : &tmW1_r;
        // weights of a routed expert whose rows fit one M-tile are read exactly once: let them leave L2 first
        const bool stream_w = ti.seg == 0 && ti.single;
        const int x_row = ti.row0 + ti.group_local * sg.a_group_stride;
        const int w_y0 = ti.group_local * sg.b_rows_per_group + ti.nb * (MODE == 0 ? 128 : 256);
        const int w_y1 = MODE == 0 ? w_y0 : w_y0 + 128;
        const int kb_half = sg.k_blocks >> 1;
        for (int kb = 0; kb < sg.k_blocks; ++kb) {
          if (kb == kb_half) *prod_half = (int)it + 1;     // the scheduler may now claim the next tile
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, budget)) { ok = false; break; }
          if (issued == p.test_withhold_stage) {
            // Self-test hook (fmmoe_test_expire_wait): the producer stops here, before it has issued any copy
            // or arrival for this stage.  Nothing will ever complete the stage's barrier, so the issuer's
            // bounded wait runs out and the CTA leaves through its tear-down path.
            stop = true;
            break;
          }
          ++issued;
          unsigned char* sW = smem + stage * S_STAGE_BYTES;
          mbar_arrive_expect_tx(&full_bar[stage], 2u * L::W_RAW + x_bytes);
          // the weight maps count columns in elements: bf16 elements, or FP8 bytes
          if (stream_w) {
            tma_load_2d_hint(sW, mW0, &full_bar[stage], kb * S_BK, w_y0, pol_stream);
            tma_load_2d_hint(sW + L::W_RAW, mW1, &full_bar[stage], kb * S_BK, w_y1, pol_stream);
          } else {
            tma_load_2d(sW, mW0, &full_bar[stage], kb * S_BK, w_y0);
            tma_load_2d(sW + L::W_RAW, mW1, &full_bar[stage], kb * S_BK, w_y1);
          }
          tma_load_2d(sW + L::X_OFF, mX, &full_bar[stage], kb * S_BK, x_row);
          if (++stage == S_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------ tile scheduler
    // Claims tiles from the global counter, decodes them (a global read of the M-tile list and a few
    // divisions) and publishes them through the slot ring: tile n+1 is claimed when the producer is half-way
    // through tile n.  Keeping this off the producer matters: its ring holds about as much work as a load takes
    // to arrive, so any pause of the producer starves the MMAs.
    if (lane == 0) {
      bool ok = true;
      for (uint32_t seq = 0; ok; ++seq) {
        if (seq >= 1) {
          const uint64_t t0 = global_timer_ns();
          while (*prod_half < (int)seq) {
            __nanosleep(64);
            if (*abort_flag || global_timer_ns() - t0 > budget) { ok = false; break; }
          }
          if (!ok) break;
        }
        const int raw_id = atomicAdd(p.tile_counter, 1);
        const int tile = raw_id < total_tiles ? raw_id : -1;
        TileInfo ti = {};
        if (tile >= 0) ti = decode_tile(p, tile, n_mt_r);
        const int slot = seq % G_SCHED;
        const uint32_t sph = (seq / G_SCHED) & 1;
        if (!mbar_wait(&sempty_bar[slot], sph ^ 1, abort_flag, budget)) { ok = false; break; }
        slot_store(ring + slot * G_SLOT_INTS, tile, ti);
        mbar_arrive(&sfull_bar[slot]);
        if (tile < 0) break;
      }
      // a scheduler that gave up because another role aborted records nothing: the status word has the cause
      if (!ok && !*abort_flag) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int as = 0; uint32_t aphase = 0;
      int cs = 0; uint32_t cphase = 0;
      bool ok = true;
      for (uint32_t it = 0; ok; ++it) {
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag, budget)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const int seg = ring[slot * G_SLOT_INTS + 1];
        const int rows = ring[slot * G_SLOT_INTS + 4];
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const uint32_t idesc = umma_idesc_bf16(128, n_pad_of(rows));
        const int k_blocks = p.seg[seg].k_blocks;
        if (!mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, budget)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d0 = tmem_base + as * 256, d1 = d0 + 128;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag, budget)) { ok = false; break; }
          if (WQ && !mbar_wait(&cfull_bar[cs], cphase, abort_flag, budget)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sS = smem_u32(smem + stage * S_STAGE_BYTES);
          const uint32_t sW = WQ ? smem_u32(smem + L::CVT_OFF + cs * 2 * S_W_BYTES) : sS;
          const uint64_t dw0 = umma_desc_sw128(sW);
          const uint64_t dw1 = umma_desc_sw128(sW + S_W_BYTES);
          const uint64_t dx = umma_desc_sw128(sS + L::X_OFF);
#pragma unroll
          for (int k = 0; k < S_BK / 16; ++k) {     // +32 bytes per K = 16 step inside the swizzle atom
            umma_bf16(d0, dw0 + 2 * k, dx + 2 * k, idesc, (kb | k) != 0);
            umma_bf16(d1, dw1 + 2 * k, dx + 2 * k, idesc, (kb | k) != 0);
          }
          umma_commit(&empty_bar[stage]);   // stage reusable once these MMAs have read it
          if (++stage == S_STAGES) { stage = 0; phase ^= 1; }
          if (WQ) {
            umma_commit(&cempty_bar[cs]);   // and so is the buffer of expanded weights
            if (++cs == S_CVT_STAGES) { cs = 0; cphase ^= 1; }
          }
        }
        if (!ok) break;
        umma_commit(&tfull_bar[as]);        // both accumulators complete
        if (++as == 2) { as = 0; aphase ^= 1; }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (WQ && warp >= 7) {
    // ------------------------------------------------------------ weight converters (FP8 stream, warps 7..14)
    // Per k-block: two boxes of 128 rows x 64 FP8 bytes (row-major, 64-byte rows) -> two boxes of 128 rows x 64
    // bf16 in the 128-byte swizzle (16-byte chunk c of row r at r*128 + ((c ^ (r & 7)) * 16)).  A thread takes
    // 16 bytes (row p/4, bytes 16*(p%4) ..) at a time: one 16-byte load, two 16-byte stores; consecutive
    // threads read consecutive pieces and the eight lanes of a quarter-warp write eight different chunks.
    const int ct = threadIdx.x - S_THREADS;      // 0 .. S_CONVERTERS-1
    int stage = 0; uint32_t phase = 0;
    int cs = 0; uint32_t cphase = 0;
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      const int slot = it % G_SCHED;
      const uint32_t sph = (it / G_SCHED) & 1;
      if (!mbar_wait(&sfull_bar[slot], sph, abort_flag, budget)) { ok = false; break; }
      const int tile = ring[slot * G_SLOT_INTS];
      const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sempty_bar[slot]);
      if (tile < 0) break;
      const Segment& sg = p.seg[ti.seg];
      // block scales of the tile's two weight boxes: lane l holds the exponent of 128-column block l
      const int n_kb128 = (sg.k_blocks + 1) >> 1;
      const int rb0 = MODE == 0 ? ti.nb : 2 * ti.nb, rb1 = MODE == 0 ? ti.nb : 2 * ti.nb + 1;
      const int rb_per_group = (sg.b_rows_per_group + 127) >> 7;
      const long long sc_base = (long long)ti.group_local * rb_per_group;
      int se0 = 0, se1 = 0;
      if (lane < n_kb128) {
        se0 = p.wscale[ti.seg][0][(sc_base + rb0) * n_kb128 + lane];
        if (rb1 < rb_per_group) se1 = p.wscale[ti.seg][1][(sc_base + rb1) * n_kb128 + lane];
      }
      for (int kb = 0; kb < sg.k_blocks; ++kb) {
        // warp-uniform outcome: the arrivals below are made by one lane on behalf of the warp
        if (!__all_sync(0xffffffffu, mbar_wait(&full_bar[stage], phase, abort_flag, budget) &&
                                     mbar_wait(&cempty_bar[cs], cphase ^ 1, abort_flag, budget))) { ok = false; break; }
        const int e0 = __shfl_sync(0xffffffffu, se0, kb >> 1), e1 = __shfl_sync(0xffffffffu, se1, kb >> 1);
        const unsigned char* raw_w = smem + stage * S_STAGE_BYTES;
        unsigned char* out_w = smem + L::CVT_OFF + cs * 2 * S_W_BYTES;
#pragma unroll
        for (int box = 0; box < 2; ++box) {
          const uint32_t mbits = (uint32_t)(247 + (box ? e1 : e0)) << 7;      // bf16 2^(120 + scale exponent)
          const uint32_t m2 = mbits | (mbits << 16);
          const __nv_bfloat162 mul = *reinterpret_cast<const __nv_bfloat162*>(&m2);
          uint4 q[S_CVT_PIECES];
#pragma unroll
          for (int i = 0; i < S_CVT_PIECES; ++i)
            q[i] = *reinterpret_cast<const uint4*>(raw_w + box * S_WQ_BYTES + (i * S_CONVERTERS + ct) * 16);
#pragma unroll
          for (int i = 0; i < S_CVT_PIECES; ++i) {
            const int pce = i * S_CONVERTERS + ct, r = pce >> 2, c = pce & 3;
            const uint32_t w4[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
            uint32_t o[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) { o[2 * j] = e4m3x2_to_bf16x2(w4[j], 0, mul); o[2 * j + 1] = e4m3x2_to_bf16x2(w4[j], 1, mul); }
            unsigned char* row = out_w + box * S_W_BYTES + r * 128;
            *reinterpret_cast<uint4*>(row + (((2 * c) ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(row + (((2 * c + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
          }
        }
        fence_proxy_async_smem();            // the MMA reads these generic-proxy writes through the async proxy
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&cfull_bar[cs]);
          mbar_arrive(&empty_bar[stage]);    // this warp is done with the stage's weight bytes
        }
        if (++stage == S_STAGES) { stage = 0; phase ^= 1; }
        if (++cs == S_CVT_STAGES) { cs = 0; cphase ^= 1; }
      }
    }
    if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                 // TMEM lane quarter this warp may access = features 32q .. 32q+31
    int as = 0; uint32_t aphase = 0;
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      const int slot = it % G_SCHED;
      const uint32_t sph = (it / G_SCHED) & 1;
      if (!mbar_wait(&sfull_bar[slot], sph, abort_flag, budget)) { ok = false; break; }
      const int tile = ring[slot * G_SLOT_INTS];
      const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sempty_bar[slot]);
      if (tile < 0) break;
      const Segment& sg = p.seg[ti.seg];
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, budget)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + as * 256 + (static_cast<uint32_t>(q * 32) << 16);
      const long long out_row0 = (long long)ti.row0 + (long long)ti.group_local * sg.out_group_stride;
      const int n_chunks = (ti.rows + 31) >> 5;
      if (MODE == 0) {
        const int feat = ti.nb * 128 + q * 32 + lane;
        const bool f_ok = feat < sg.n_valid;
        __nv_bfloat16* dst = p.act[ti.seg] + out_row0 * sg.ld_out + feat;
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
          uint32_t g[32], u[32];
          tmem_ld32(taddr + c * 32, g);
          tmem_ld32(taddr + 128 + c * 32, u);
          tmem_ld_wait();
          const int nt = min(32, ti.rows - c * 32);      // warp-uniform
          if (f_ok) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < nt) {
                const float g0 = __uint_as_float(g[j]);
                const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(u[j]);
                dst[(long long)(c * 32 + j) * sg.ld_out] = __float2bfloat16_rn(a0);   // 32 lanes: 64 contiguous bytes
              }
            }
          }
        }
      } else {
        const int feat0 = ti.nb * 256 + q * 32 + lane;
        const bool f0_ok = feat0 < sg.n_valid, f1_ok = feat0 + 128 < sg.n_valid;
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
          const int nt = min(32, ti.rows - c * 32);      // warp-uniform
          int tok_l = 0; float gate_l = 1.f;
          if (ti.seg == 0) {
            if (lane < nt) { tok_l = p.row_token[ti.row0 + c * 32 + lane]; gate_l = p.row_gate[ti.row0 + c * 32 + lane]; }
          } else {
            tok_l = ti.row0 + c * 32 + lane;
          }
          if (p.deterministic) gate_l = 1.f;   // gates are applied by the ordered gather
          uint32_t v0[32], v1[32];
          tmem_ld32(taddr + c * 32, v0);
          tmem_ld32(taddr + 128 + c * 32, v1);
          tmem_ld_wait();
          if (p.pair) {
            // pair-row mode: gate-scaled bf16 rows per pair; for one token the warp writes 64 contiguous bytes
            __nv_bfloat16* yp = p.yb[ti.seg] + (out_row0 + c * 32) * sg.ld_out + feat0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float gt = __shfl_sync(0xffffffffu, gate_l, j);
              if (j < nt) {
                if (f0_ok) yp[(long long)j * sg.ld_out] = __float2bfloat16_rn(gt * __uint_as_float(v0[j]));
                if (f1_ok) yp[(long long)j * sg.ld_out + 128] = __float2bfloat16_rn(gt * __uint_as_float(v1[j]));
              }
            }
          } else if (p.deterministic) {
            float* yb = p.y[ti.seg] + (out_row0 + c * 32) * sg.ld_out + feat0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < nt) {
                if (f0_ok) yb[(long long)j * sg.ld_out] = __uint_as_float(v0[j]);
                if (f1_ok) yb[(long long)j * sg.ld_out + 128] = __uint_as_float(v1[j]);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int tk = __shfl_sync(0xffffffffu, tok_l, j);
              const float gt = __shfl_sync(0xffffffffu, gate_l, j);
              if (j < nt) {
                float* ab = p.acc + (long long)tk * sg.ld_out + feat0;       // the warp adds 128 contiguous bytes
                if (f0_ok) red_add_f32(ab, gt * __uint_as_float(v0[j]));
                if (f1_ok) red_add_f32(ab + 128, gt * __uint_as_float(v1[j]));
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&tempty_bar[as]);
      if (++as == 2) { as = 0; aphase ^= 1; }
    }
    if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
  }

  // ---------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies still in flight time to land before the shared memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, S_TMEM_COLS);
  }
}

// ---------------------------------------------------------------- host side
template <int WQ>
static fmmoe_status launch_ffn_sm_impl(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s) {
  using L = SmLayout<WQ>;
  const fmmoe_layer_desc& d = *a.d;
  const int H = d.hidden, I = d.inter, E = d.n_experts, Ns = d.n_shared, Is = d.shared_inter;
  if (!h->encode_tiled) return FMMOE_ERR_CUDA;
  if (a.T == 0) return FMMOE_OK;
  const int mtps = (int)((a.T + TC_BLOCK_M - 1) / TC_BLOCK_M);
  const uint64_t p_rows = (uint64_t)a.p_max;

  CUtensorMap X1r[4], X2r[4], X1s, X2s, G1r, U1r, G1s, U1s, D2r, D2s;
  bool ok = true;
  for (int i = 0; i < 4; ++i) {
    ok &= make_map(h, &X1r[i], a.xp, p_rows, H, 32 * (i + 1));
    ok &= make_map(h, &X2r[i], a.act, p_rows, I, 32 * (i + 1));
  }
  auto wmap = [&](CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols) {
    return WQ ? make_map_u8(h, m, base, rows, cols, 128) : make_map(h, m, base, rows, cols, 128);
  };
  ok &= wmap(&G1r, a.w->w_gate, (uint64_t)E * I, H);
  ok &= wmap(&U1r, a.w->w_up, (uint64_t)E * I, H);
  ok &= wmap(&D2r, a.w->w_down, (uint64_t)E * H, I);
  if (Ns) {
    ok &= make_map(h, &X1s, a.x, (uint64_t)a.T, H, 128);
    ok &= wmap(&G1s, a.w->ws_gate, (uint64_t)Ns * Is, H);
    ok &= wmap(&U1s, a.w->ws_up, (uint64_t)Ns * Is, H);
    ok &= make_map(h, &X2s, a.act_sh, (uint64_t)Ns * a.T, Is, 128);
    ok &= wmap(&D2s, a.w->ws_down, (uint64_t)Ns * H, Is);
  } else {
    X1s = X1r[3]; G1s = G1r; U1s = U1r; X2s = X2r[3]; D2s = D2r;   // never dereferenced without shared experts
  }
  if (!ok) return FMMOE_ERR_CUDA;

  GemmParams p1 = {};
  p1.mtiles = a.mtiles; p1.n_mtiles = a.n_mtiles; p1.max_mtiles = a.max_mtiles;
  p1.block_m = TC_BLOCK_M; p1.shared_mtiles = Ns * mtps; p1.mt_per_shared = mtps; p1.T = a.T;
  p1.seg[0] = Segment{(I + 127) / 128, H / S_BK, I, I, 0, 0, I};
  p1.seg[1] = Segment{Ns ? (Is + 127) / 128 : 0, H / S_BK, Is, Is, 0, (int)a.T, Is};
  p1.act[0] = static_cast<__nv_bfloat16*>(a.act); p1.act[1] = static_cast<__nv_bfloat16*>(a.act_sh);
  p1.status = a.d_status;
  p1.x = static_cast<const __nv_bfloat16*>(a.x); p1.ld_x = H; p1.row_token = a.row_token; p1.gather = 0;
  p1.tile_counter = a.tile_counters;
  p1.wait_budget_ns = h->wait_budget_ns; p1.test_withhold_stage = a.test_withhold_stage;
  p1.wscale[0][0] = a.w->w_gate_scale; p1.wscale[0][1] = a.w->w_up_scale;
  p1.wscale[1][0] = a.w->ws_gate_scale; p1.wscale[1][1] = a.w->ws_up_scale;

  GemmParams p2 = p1;
  p2.seg[0] = Segment{(H + 255) / 256, I / S_BK, H, H, 0, 0, H};
  p2.seg[1] = Segment{Ns ? (H + 255) / 256 : 0, Ns ? Is / S_BK : 0, H, H, (int)a.T, (int)a.T, H};
  p2.row_token = a.row_token; p2.row_gate = a.row_gate; p2.acc = a.acc;
  p2.y[0] = a.y; p2.y[1] = a.ysh; p2.deterministic = a.deterministic;
  p2.yb[0] = static_cast<__nv_bfloat16*>(a.yb); p2.yb[1] = static_cast<__nv_bfloat16*>(a.ybsh); p2.pair = a.pair;
  p2.tile_counter = a.tile_counters + 1;
  p2.test_withhold_stage = -1;
  p2.wscale[0][0] = p2.wscale[0][1] = a.w->w_down_scale;
  p2.wscale[1][0] = p2.wscale[1][1] = a.w->ws_down_scale;

  bool& attr_set = WQ ? h->smq_attr_set : h->sm_attr_set;
  if (!attr_set) {
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_sm_kernel<0, WQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM_BYTES));
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_sm_kernel<1, WQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM_BYTES));
    attr_set = true;
  }
  const int grid = a.grid_override > 0 ? a.grid_override : h->sm_count;
  { ProfScope ps(h, FMMOE_KERNEL_GEMM1, s); FMMOE_CUDA_TRY(launch_pdl(ffn_sm_kernel<0, WQ>, dim3(grid), dim3(L::THREADS), L::SMEM_BYTES, s, 1, X1r[0], X1r[1], X1r[2], X1r[3], X1s, G1r, U1r, G1s, U1s, p1)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  { ProfScope ps(h, FMMOE_KERNEL_GEMM2, s); FMMOE_CUDA_TRY(launch_pdl(ffn_sm_kernel<1, WQ>, dim3(grid), dim3(L::THREADS), L::SMEM_BYTES, s, 1, X2r[0], X2r[1], X2r[2], X2r[3], X2s, D2r, D2r, D2s, D2s, p2)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 2;
  return FMMOE_OK;
}

fmmoe_status launch_ffn_sm(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s) {
  return a.d->weight_format == FMMOE_WEIGHTS_FP8_BLOCK128 ? launch_ffn_sm_impl<1>(h, a, s) : launch_ffn_sm_impl<0>(h, a, s);
}

}  // namespace fmmoe
