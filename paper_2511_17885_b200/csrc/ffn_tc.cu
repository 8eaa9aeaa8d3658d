// Expert FFNs on the 5th-generation tensor cores (tcgen05), bf16 in / fp32 accumulate.
//
// Eq. 4 needs, for every routed (token, expert) pair and every (token, shared expert)
// pair, y = W_down (silu(W_gate x) * (W_up x)).  With the pairs grouped by expert
// this is two grouped GEMMs:
//   GEMM-1  [rows_e, H] x [H, 2*S_m]  -> SwiGLU in the epilogue -> act [rows, S_m] bf16
//   GEMM-2  [rows_e, S_m] x [S_m, H]  -> gate-weighted combine in the epilogue
// Both run in one persistent, warp-specialised kernel template:
//   warp 0    : TMA producer (A tile 128x64 + two B boxes 128x64 per stage, 128B swizzle, L2 eviction hints)
//   warp 6    : tile scheduler (claims and decodes tiles one ahead of the producer)
//   warps 7-10: GEMM-1 (from 256 tokens on by default): gather the rows of a routed M-tile straight
//               from x by token with cp.async into the same swizzled layout, so that no
//               expert-ordered copy of x is written and read back (measured 3-12 % of a step faster
//               than the copy plus plain TMA boxes between 2,432 and 14,336 tokens; with the copy
//               the kernel is launched without these warps)
//   warp 1    : UMMA issuer   (one thread; 128x256x16 tcgen05.mma, accumulators in TMEM)
//   warps 2-5 : epilogue      (tcgen05.ld -> registers -> shared-memory transpose -> coalesced
//               global stores / reductions), overlapped with the next tile's main loop
//               through two TMEM accumulator stages (2 x 256 columns).
// A tile is (M-tile of 128 grouped rows) x (N-block).  Tiles are handed out dynamically (an
// atomic counter; the scheduler warp publishes each tile, decoded, to the other roles through a
// small shared-memory ring), in an order that
//   - walks the routed tiles M-tile-major, so the 128 activation rows of an M-tile are
//     re-read from L2 by CTAs running at the same time while every weight tile streams
//     from HBM once,
//   - walks the shared-expert tiles N-block-major, so the CTAs running at the same time
//     share one weight tile, and
//   - interleaves the two kinds evenly: at small batch routed tiles are bound by the
//     weight stream and shared-expert tiles by the tensor pipe, and mixing them keeps both
//     busy.
// GEMM-1's B tile is 128 gate rows + 128 up rows of the same expert, so one thread
// holds gate and up of the same (row, column) in TMEM columns c and 128+c.
// Every wait is bounded; on expiry the CTA records FMMOE_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"
#include "ffn_common.cuh"

namespace fmmoe {

constexpr int G_BM = TC_BLOCK_M;   // 128
constexpr int G_BK = 64;           // one 128-byte swizzle atom of bf16
constexpr int G_STAGES = 4;
constexpr int G_A_BYTES = G_BM * G_BK * 2;          // 16 KB
constexpr int G_B_BYTES = 2 * 128 * G_BK * 2;       // 32 KB (two 128-row boxes)
constexpr int G_STAGE_BYTES = G_A_BYTES + G_B_BYTES;
constexpr int G_THREADS = 224;          // producer warp, issuer warp, four epilogue warps, tile-scheduler warp
constexpr int G_LOADERS = 128;          // GEMM-1 only: four more warps that gather the routed rows of x
constexpr int G_THREADS_G1 = G_THREADS + G_LOADERS;
constexpr int G_TMEM_COLS = 512;
constexpr int G_SMEM_BYTES = G_STAGES * G_STAGE_BYTES + G_EPI_BYTES + 1024 /*align*/ + 384 /*barriers, tile ring*/;

// MODE 0: GEMM-1 + SwiGLU.  MODE 1: GEMM-2 + combine.
template <int MODE>
__global__ void __launch_bounds__(MODE == 0 ? G_THREADS_G1 : G_THREADS, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tmA_r, const __grid_constant__ CUtensorMap tmA_s,
              const __grid_constant__ CUtensorMap tmB0_r, const __grid_constant__ CUtensorMap tmB1_r,
              const __grid_constant__ CUtensorMap tmB0_s, const __grid_constant__ CUtensorMap tmB1_s,
              const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + ((1024 - (raw & 1023)) & 1023);   // 1024-byte aligned tiles (128B swizzle)
  float* epi = reinterpret_cast<float*>(smem + G_STAGES * G_STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G_STAGES * G_STAGE_BYTES + G_EPI_BYTES);
  uint64_t* full_bar = bars;                   // [G_STAGES]
  uint64_t* empty_bar = bars + G_STAGES;       // [G_STAGES]
  uint64_t* tfull_bar = bars + 2 * G_STAGES;   // [2]
  uint64_t* tempty_bar = tfull_bar + 2;        // [2]
  uint64_t* sfull_bar = tempty_bar + 2;        // [G_SCHED]
  uint64_t* sempty_bar = sfull_bar + G_SCHED;  // [G_SCHED]
  volatile int* ring = reinterpret_cast<volatile int*>(sempty_bar + G_SCHED);   // [G_SCHED][G_SLOT_INTS]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ring) + G_SCHED * G_SLOT_INTS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* prod_half = abort_flag + 1;    // tiles the producer has taken half-way (paces the tile scheduler)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    // GEMM-1: a stage is full when the producer's TMA bytes have landed AND every loader thread's copies have
    for (int i = 0; i < G_STAGES; ++i) { mbar_init(&full_bar[i], (MODE == 0 && p.gather) ? 1 + G_LOADERS : 1); mbar_init(&empty_bar[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull_bar[i], 1); mbar_init(&tempty_bar[i], 128); }
    // readers of a tile id: producer + issuer + 4 epilogue warps (+ 4 loader warps in GEMM-1)
    for (int i = 0; i < G_SCHED; ++i) { mbar_init(&sfull_bar[i], 1); mbar_init(&sempty_bar[i], (MODE == 0 && p.gather) ? 10 : 6); }
    *abort_flag = 0;
    *prod_half = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, G_TMEM_COLS);
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
      tma_prefetch_desc(&tmA_r);
      tma_prefetch_desc(&tmB0_r); tma_prefetch_desc(&tmB1_r);
      if (p.shared_mtiles) { tma_prefetch_desc(&tmA_s); tma_prefetch_desc(&tmB0_s); tma_prefetch_desc(&tmB1_s); }
      const uint64_t pol_stream = l2_policy_evict_first();
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (uint32_t it = 0; ok; ++it) {
        // the tile comes decoded from the scheduler warp: the producer touches no global memory but the TMA maps
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const Segment& sg = p.seg[ti.seg];
        const CUtensorMap* mA = ti.seg ? &tmA_s : &tmA_r;
        const CUtensorMap* mB0 = ti.seg ? &tmB0_s : &tmB0_r;
        const CUtensorMap* mB1 = ti.seg ? &tmB1_s : &tmB1_r;
        // Weights of a routed expert whose rows fit one M-tile are read exactly once: let them
        // leave L2 first.  Everything that is re-read (weights of multi-tile experts and of the
        // shared experts, activation tiles) keeps the default priority: tiles that share data
        // are adjacent in the order, so plain LRU keeps it resident for as long as it is needed.
        const bool stream_b = ti.seg == 0 && ti.single;
        // GEMM-1 reads a routed M-tile's rows straight from x through the token list (loader warps,
        // cp.async): the TMA engine, whose row rate bounds the weight stream, carries weights only
        const bool gather_a = MODE == 0 && p.gather && ti.seg == 0;
        const int a_row = ti.row0 + ti.group_local * sg.a_group_stride;
        const int b_y0 = ti.group_local * sg.b_rows_per_group + ti.nb * (MODE == 0 ? 128 : 256);
        const int b_y1 = MODE == 0 ? b_y0 : b_y0 + 128;
        const int kb_half = sg.k_blocks >> 1;
        for (int kb = 0; kb < sg.k_blocks; ++kb) {
          if (kb == kb_half) *prod_half = (int)it + 1;     // the scheduler may now claim the next tile
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * G_STAGE_BYTES;
          mbar_arrive_expect_tx(&full_bar[stage], gather_a ? G_B_BYTES : G_STAGE_BYTES);
          if (!gather_a) tma_load_2d(sA, mA, &full_bar[stage], kb * G_BK, a_row);
          if (stream_b) {
            tma_load_2d_hint(sA + G_A_BYTES, mB0, &full_bar[stage], kb * G_BK, b_y0, pol_stream);
            tma_load_2d_hint(sA + G_A_BYTES + G_B_BYTES / 2, mB1, &full_bar[stage], kb * G_BK, b_y1, pol_stream);
          } else {
            tma_load_2d(sA + G_A_BYTES, mB0, &full_bar[stage], kb * G_BK, b_y0);
            tma_load_2d(sA + G_A_BYTES + G_B_BYTES / 2, mB1, &full_bar[stage], kb * G_BK, b_y1);
          }
          if (++stage == G_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------ tile scheduler
    // Claims tiles from the global counter, decodes them (a global read of the M-tile list and a few
    // divisions) and publishes them through the slot ring, one tile ahead of the producer: tile n+1 is
    // claimed when the producer is half-way through tile n.  Keeping this off the producer matters: its
    // ring holds about as much work as a load takes to arrive, so any pause of the producer starves the MMAs.
    if (lane == 0) {
      bool ok = true;
      for (uint32_t seq = 0; ok; ++seq) {
        if (seq >= 1) {     // tile n+1 is claimed once the producer is half-way through tile n
          const uint64_t t0 = global_timer_ns();
          while (*prod_half < (int)seq) {
            __nanosleep(64);
            if (*abort_flag || global_timer_ns() - t0 > 2000000000ull) { ok = false; break; }
          }
          if (!ok) break;
        }
        const int raw_id = atomicAdd(p.tile_counter, 1);
        const int tile = raw_id < total_tiles ? raw_id : -1;
        TileInfo ti = {};
        if (tile >= 0) ti = decode_tile(p, tile, n_mt_r);
        const int slot = seq % G_SCHED;
        const uint32_t sph = (seq / G_SCHED) & 1;
        if (!mbar_wait(&sempty_bar[slot], sph ^ 1, abort_flag)) { ok = false; break; }
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
      // A tile with at most 64 valid rows runs as M = 64 MMAs: same duration, half the datapaths
      // switching (at batch 1 the GPU sits at its power cap, where that buys clock)
      constexpr uint32_t idesc128 = umma_idesc_bf16(G_BM, 256), idesc64 = umma_idesc_bf16(64, 256);
      int stage = 0; uint32_t phase = 0;
      int as = 0; uint32_t aphase = 0;
      bool ok = true;
      for (uint32_t it = 0; ok; ++it) {
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const int seg = ring[slot * G_SLOT_INTS + 1];
        const uint32_t idesc = ring[slot * G_SLOT_INTS + 4] <= 64 ? idesc64 : idesc128;
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const int k_blocks = p.seg[seg].k_blocks;
        if (!mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * 256;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
          if (MODE == 0 && p.gather) fence_proxy_async_smem();   // rows written by the loader warps' cp.async
          tc_fence_after();
          const uint32_t sA = smem_u32(smem + stage * G_STAGE_BYTES);
          const uint64_t da = umma_desc_sw128(sA);
          const uint64_t db = umma_desc_sw128(sA + G_A_BYTES);
#pragma unroll
          for (int k = 0; k < G_BK / 16; ++k)
            umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);   // +32 bytes per K=16 step
          umma_commit(&empty_bar[stage]);   // stage reusable once these MMAs have read it
          if (++stage == G_STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        umma_commit(&tfull_bar[as]);        // accumulator complete
        if (++as == 2) { as = 0; aphase ^= 1; }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp >= 7) {
    // ------------------------------------------------------------ row loaders (GEMM-1 only, warps 7..10)
    // Every stage of a routed tile: 128 rows x 128 bytes of x, row r = token row_token[row0 + r],
    // written where a TMA box with the 128-byte swizzle would put them (16-byte chunk c of row r at
    // r*128 + ((c ^ (r & 7)) * 16)).  Eight lanes cover one row, a thread serves rows q, q+16, ...
    // For other tiles the loaders only keep the stage barriers in step.
    if (MODE == 0 && p.gather) {
      const int lt = threadIdx.x - G_THREADS;      // 0..127
      const int chunk = lt & 7, rq = lt >> 3;      // rq 0..15
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      const __nv_bfloat16* xg = p.x;
      for (uint32_t it = 0; ok; ++it) {
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const Segment& sg = p.seg[ti.seg];
        const bool gather_a = ti.seg == 0;
        const __nv_bfloat16* src[8];
        uint32_t dst_off[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = rq + 16 * i;
          const bool valid = gather_a && r < ti.rows;
          const long long tok = valid ? p.row_token[ti.row0 + r] : -1;
          src[i] = valid ? xg + tok * p.ld_x + chunk * 8 : nullptr;
          dst_off[i] = (uint32_t)(r * 128 + ((chunk ^ (r & 7)) << 4));
        }
        for (int kb = 0; kb < sg.k_blocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          if (gather_a) {
            const uint32_t sA = smem_u32(smem + stage * G_STAGE_BYTES);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (src[i]) cp_async_16(sA + dst_off[i], src[i] + kb * G_BK);
            cp_async_arrive_noinc(&full_bar[stage]);
          } else {
            mbar_arrive(&full_bar[stage]);
          }
          if (++stage == G_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                 // TMEM lane quarter this warp may access
    float* stg = epi + q * 32 * G_EPI_LD;   // this warp's 32 x 32 transpose block
    int as = 0; uint32_t aphase = 0;
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      const int slot = it % G_SCHED;
      const uint32_t sph = (it / G_SCHED) & 1;
      if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
      const int tile = ring[slot * G_SLOT_INTS];
      const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sempty_bar[slot]);
      if (tile < 0) break;
      const Segment& sg = p.seg[ti.seg];
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + as * 256 + (static_cast<uint32_t>(q * 32) << 16);
      // M = 128: row i of the tile sits in TMEM lane i.  M = 64 (tiles of at most 64 rows): row i sits in
      // lane 32 * (i / 16) + i % 16, so each warp's lane quarter holds 16 rows in its lanes 0..15.
      const int rpw = ti.rows <= 64 ? 16 : 32;          // rows per warp
      tc_epilogue<MODE>(p, ti, sg, taddr, stg, lane, q, rpw);
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
    tmem_dealloc(tmem_base, G_TMEM_COLS);
  }
}

// ---------------------------------------------------------------- host side
fmmoe_status launch_ffn_tc(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s) {
  const fmmoe_layer_desc& d = *a.d;
  const int H = d.hidden, I = d.inter, E = d.n_experts, Ns = d.n_shared, Is = d.shared_inter;
  if (!h->encode_tiled) return FMMOE_ERR_CUDA;
  if (a.T == 0) return FMMOE_OK;
  const int mtps = (int)((a.T + G_BM - 1) / G_BM);
  const uint64_t p_rows = (uint64_t)a.p_max;

  CUtensorMap A1s, G1r, U1r, G1s, U1s, A2r, A2s, D2r, D2s;
  bool ok = true;
  CUtensorMap A1r;
  ok &= make_map(h, &A1r, a.gather_in_gemm ? a.x : a.xp, a.gather_in_gemm ? (uint64_t)a.T : p_rows, H, 128);
  ok &= make_map(h, &G1r, a.w->w_gate, (uint64_t)E * I, H, 128);
  ok &= make_map(h, &U1r, a.w->w_up, (uint64_t)E * I, H, 128);
  ok &= make_map(h, &A2r, a.act, p_rows, I, 128);
  ok &= make_map(h, &D2r, a.w->w_down, (uint64_t)E * H, I, 128);
  if (Ns) {
    ok &= make_map(h, &A1s, a.x, (uint64_t)a.T, H, 128);
    ok &= make_map(h, &G1s, a.w->ws_gate, (uint64_t)Ns * Is, H, 128);
    ok &= make_map(h, &U1s, a.w->ws_up, (uint64_t)Ns * Is, H, 128);
    ok &= make_map(h, &A2s, a.act_sh, (uint64_t)Ns * a.T, Is, 128);
    ok &= make_map(h, &D2s, a.w->ws_down, (uint64_t)Ns * H, Is, 128);
  } else {
    A1s = G1r; G1s = G1r; U1s = U1r; A2s = A2r; D2s = D2r;   // never dereferenced without shared experts
  }
  if (!ok) return FMMOE_ERR_CUDA;

  GemmParams p1 = {};
  p1.mtiles = a.mtiles; p1.n_mtiles = a.n_mtiles; p1.max_mtiles = a.max_mtiles;
  p1.block_m = G_BM; p1.shared_mtiles = Ns * mtps; p1.mt_per_shared = mtps; p1.T = a.T;
  p1.seg[0] = Segment{(I + 127) / 128, H / G_BK, I, I, 0, 0, I};
  p1.seg[1] = Segment{Ns ? (Is + 127) / 128 : 0, H / G_BK, Is, Is, 0, (int)a.T, Is};
  p1.act[0] = static_cast<__nv_bfloat16*>(a.act); p1.act[1] = static_cast<__nv_bfloat16*>(a.act_sh);
  p1.status = a.d_status;
  p1.x = static_cast<const __nv_bfloat16*>(a.x); p1.ld_x = H; p1.row_token = a.row_token; p1.gather = a.gather_in_gemm;
  p1.tile_counter = a.tile_counters;

  GemmParams p2 = p1;
  p2.seg[0] = Segment{(H + 255) / 256, I / G_BK, H, H, 0, 0, H};
  p2.seg[1] = Segment{Ns ? (H + 255) / 256 : 0, Ns ? Is / G_BK : 0, H, H, (int)a.T, (int)a.T, H};
  p2.row_token = a.row_token; p2.row_gate = a.row_gate; p2.acc = a.acc;
  p2.y[0] = a.y; p2.y[1] = a.ysh; p2.deterministic = a.deterministic;
  p2.yb[0] = static_cast<__nv_bfloat16*>(a.yb); p2.yb[1] = static_cast<__nv_bfloat16*>(a.ybsh); p2.pair = a.pair;
  p2.tile_counter = a.tile_counters + 1;

  if (!h->tc_attr_set) {
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES));
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES));
    h->tc_attr_set = true;
  }
  const int grid = h->sm_count;
  { ProfScope ps(h, FMMOE_KERNEL_GEMM1, s); FMMOE_CUDA_TRY(launch_pdl(ffn_tc_kernel<0>, dim3(grid), dim3(a.gather_in_gemm ? G_THREADS_G1 : G_THREADS), G_SMEM_BYTES, s, 1, A1r, A1s, G1r, U1r, G1s, U1s, p1)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  { ProfScope ps(h, FMMOE_KERNEL_GEMM2, s); FMMOE_CUDA_TRY(launch_pdl(ffn_tc_kernel<1>, dim3(grid), dim3(G_THREADS), G_SMEM_BYTES, s, 1, A2r, A2s, D2r, D2r, D2s, D2s, p2)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 2;
  return FMMOE_OK;
}

}  // namespace fmmoe
