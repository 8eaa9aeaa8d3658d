// Expert FFNs on the tcgen05 tensor cores with CTA pairs (cta_group::2), for batches whose experts hold
// several hundred rows.
//
// At that size the grouped GEMMs of Eq. 4 are a dense contraction.  A single CTA computing a 128 x 256 tile brings
// 48 KB into shared memory per 64-deep k-block (128 rows of activations, 256 rows of weights) for 512
// tensor-core cycles of work, 96 bytes per cycle if the pipe were to stay busy; the one-CTA kernel is measured
// at 62-79 B/clk/SM with the tensor pipe 67-84 % busy.  Two CTAs of a cluster that share one MMA of M = 256
// halve the weight traffic: each loads its own 128 activation rows and HALF of the 256 weight rows, 32 KB per
// k-block, and its ring holds six stages instead of four.
//
//   cluster rank r (0 = leader, 1 = partner), tile = (256 grouped rows of one expert) x (256 output columns):
//     A  rows  row0 + 128 r .. + 127 of the tile                      (own shared memory, own TMA loads)
//     B  GEMM-1: r = 0 the 128 gate rows, r = 1 the 128 up rows of the expert's column block
//        GEMM-2: rows 128 r .. 128 r + 127 of the 256-row block of W_down
//     D  rows 128 r .. of the 256 x 256 accumulator, in the CTA's own tensor memory: [gate | up] columns as in
//        the one-CTA kernel, so the epilogue is that kernel's, run by both CTAs on their own rows.
//   Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (leader only; both CTAs' warp 1 allocate tensor
//   memory), warps 2-5 epilogue, warp 6 tile scheduler.  Tiles are assigned statically (cluster c takes tiles
//   c, c + clusters, ...: every tile of a launch has the same k extent), so both CTAs derive the same sequence
//   without talking to each other.
//   Barriers: the partner's TMA loads credit their bytes to the LEADER's full barrier; the leader's commit
//   arrives on both CTAs' empty / accumulator-full barriers (multicast commit: no data is multicast anywhere);
//   the partner's epilogue warps arrive on the leader's accumulator-empty barrier through the cluster.
// Every wait is bounded; on expiry the CTA records FMMOE_ERR_TIMEOUT and leaves (its partner's waits then run
// out too), and both still meet at the cluster barriers of the tear-down.
//
// Status: optional (FMMOE_CTA_PAIR_MIN_TOKENS), off by default.  Measured on the batch of four Qwen3-MoE-style
// sequences it is no faster than the one-CTA kernel (GEMM-1 354-364 us against 354-379 us, GEMM-2 277-288 us
// against 243-265 us, plus the expert-ordered copy of x that it reads instead of gathering rows itself): at that
// size the GPU sits at its power cap, where halving the shared-memory intake buys little.  The kernels are
// launched in plain stream order: launched with programmatic dependent launch, a run of a few hundred steps
// stalled in one of the hardware waits that cannot be bounded (cluster barrier, pair allocation, grid
// dependency); in stream order 3,000 steps in a row and the benchmark ran clean.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"
#include "ffn_common.cuh"

namespace fmmoe {

constexpr int P_BK = 64;
constexpr int P_STAGES = 6;
constexpr int P_A_BYTES = 128 * P_BK * 2;          // 16 KB: this CTA's 128 activation rows
constexpr int P_B_BYTES = 128 * P_BK * 2;          // 16 KB: this CTA's half of the weight tile
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES;
constexpr int P_THREADS = 224;
constexpr int P_TMEM_COLS = 512;
constexpr int P_SMEM_BYTES = P_STAGES * P_STAGE_BYTES + G_EPI_BYTES + 1024 /*align*/ + 512 /*barriers, tile ring*/;

template <int MODE>
__global__ void __launch_bounds__(P_THREADS, 1)
ffn_tc2_kernel(const __grid_constant__ CUtensorMap tmA_r, const __grid_constant__ CUtensorMap tmA_s,
               const __grid_constant__ CUtensorMap tmB0_r, const __grid_constant__ CUtensorMap tmB1_r,
               const __grid_constant__ CUtensorMap tmB0_s, const __grid_constant__ CUtensorMap tmB1_s,
               const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + ((1024 - (raw & 1023)) & 1023);   // the same offset in both CTAs of the pair
  float* epi = reinterpret_cast<float*>(smem + P_STAGES * P_STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P_STAGES * P_STAGE_BYTES + G_EPI_BYTES);
  uint64_t* full_bar = bars;                   // [P_STAGES]  used in the leader: both CTAs' bytes of a stage
  uint64_t* empty_bar = bars + P_STAGES;       // [P_STAGES]  per CTA: the MMAs have read this CTA's stage
  uint64_t* tfull_bar = bars + 2 * P_STAGES;   // [2]         per CTA: accumulator stage complete
  uint64_t* tempty_bar = tfull_bar + 2;        // [2]         used in the leader: both CTAs' epilogues have drained it
  uint64_t* sfull_bar = tempty_bar + 2;        // [G_SCHED]
  uint64_t* sempty_bar = sfull_bar + G_SCHED;  // [G_SCHED]
  volatile int* ring = reinterpret_cast<volatile int*>(sempty_bar + G_SCHED);   // [G_SCHED][G_SLOT_INTS]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ring) + G_SCHED * G_SLOT_INTS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();           // 0: leader, 1: partner
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < P_STAGES; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
    // accumulator-empty: one arrival per epilogue warp of both CTAs
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull_bar[i], 1); mbar_init(&tempty_bar[i], 8); }
    // readers of a tile: producer + 4 epilogue warps (+ the issuer in the leader)
    for (int i = 0; i < G_SCHED; ++i) { mbar_init(&sfull_bar[i], 1); mbar_init(&sempty_bar[i], leader ? 6 : 5); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc_pair(tmem_slot, P_TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the partner's barriers exist before anything of this CTA can signal them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();
  const int n_mt_r = p.n_mtiles ? min(max(*p.n_mtiles, 0), p.max_mtiles) : 0;
  const int total_tiles = n_mt_r * p.seg[0].n_nblocks + p.shared_mtiles * p.seg[1].n_nblocks;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      tma_prefetch_desc(&tmA_r); tma_prefetch_desc(&tmB0_r); tma_prefetch_desc(&tmB1_r);
      if (p.shared_mtiles) { tma_prefetch_desc(&tmA_s); tma_prefetch_desc(&tmB0_s); tma_prefetch_desc(&tmB1_s); }
      uint32_t full_leader[P_STAGES];      // the leader's full barriers as cluster addresses
#pragma unroll
      for (int i = 0; i < P_STAGES; ++i) full_leader[i] = cluster_map_shared(smem_u32(&full_bar[i]), 0);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (uint32_t it = 0; ok; ++it) {
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const Segment& sg = p.seg[ti.seg];
        const CUtensorMap* mA = ti.seg ? &tmA_s : &tmA_r;
        // this CTA's half of the weight tile
        const CUtensorMap* mB = MODE == 0 ? (rank == 0 ? (ti.seg ? &tmB0_s : &tmB0_r) : (ti.seg ? &tmB1_s : &tmB1_r))
                                          : (ti.seg ? &tmB0_s : &tmB0_r);
        const int a_row = ti.row0 + 128 * (int)rank + ti.group_local * sg.a_group_stride;
        const int b_y = ti.group_local * sg.b_rows_per_group + ti.nb * (MODE == 0 ? 128 : 256) + (MODE == 0 ? 0 : 128 * (int)rank);
        for (int kb = 0; kb < sg.k_blocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * P_STAGE_BYTES;
          if (leader) mbar_arrive_expect_tx(&full_bar[stage], 2u * P_STAGE_BYTES);   // both CTAs' boxes
          tma_load_2d_pair(sA, mA, full_leader[stage], kb * P_BK, a_row);
          tma_load_2d_pair(sA + P_A_BYTES, mB, full_leader[stage], kb * P_BK, b_y);
          if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------ tile scheduler (both CTAs, the same sequence)
    if (lane == 0) {
      bool ok = true;
      for (uint32_t seq = 0; ok; ++seq) {
        const long long cand = (long long)cluster_id + (long long)seq * n_clusters;
        const int tile = cand < total_tiles ? (int)cand : -1;
        TileInfo ti = {};
        if (tile >= 0) ti = decode_tile(p, tile, n_mt_r);
        const int slot = seq % G_SCHED;
        const uint32_t sph = (seq / G_SCHED) & 1;
        if (!mbar_wait(&sempty_bar[slot], sph ^ 1, abort_flag)) { ok = false; break; }
        slot_store(ring + slot * G_SLOT_INTS, tile, ti);
        mbar_arrive(&sfull_bar[slot]);
        if (tile < 0) break;
      }
      if (!ok && !*abort_flag) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(256, 256);
      int stage = 0; uint32_t phase = 0;
      int as = 0; uint32_t aphase = 0;
      bool ok = true;
      for (uint32_t it = 0; ok; ++it) {
        const int slot = it % G_SCHED;
        const uint32_t sph = (it / G_SCHED) & 1;
        if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
        const int tile = ring[slot * G_SLOT_INTS];
        const int seg = ring[slot * G_SLOT_INTS + 1];
        mbar_arrive(&sempty_bar[slot]);
        if (tile < 0) break;
        const int k_blocks = p.seg[seg].k_blocks;
        if (!mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * 256;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sA = smem_u32(smem + stage * P_STAGE_BYTES);
          const uint64_t da = umma_desc_sw128(sA);
          const uint64_t db = umma_desc_sw128(sA + P_A_BYTES);
#pragma unroll
          for (int k = 0; k < P_BK / 16; ++k)
            umma_bf16_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          umma_commit_pair_multicast(&empty_bar[stage], 3);   // both CTAs' stage is reusable once these MMAs have read it
          if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        umma_commit_pair_multicast(&tfull_bar[as], 3);        // accumulator complete, in both CTAs
        if (++as == 2) { as = 0; aphase ^= 1; }
      }
      if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
    const int q = warp & 3;
    float* stg = epi + q * 32 * G_EPI_LD;
    uint32_t tempty_leader[2];
    tempty_leader[0] = cluster_map_shared(smem_u32(&tempty_bar[0]), 0);
    tempty_leader[1] = cluster_map_shared(smem_u32(&tempty_bar[1]), 0);
    int as = 0; uint32_t aphase = 0;
    bool ok = true;
    for (uint32_t it = 0; ok; ++it) {
      const int slot = it % G_SCHED;
      const uint32_t sph = (it / G_SCHED) & 1;
      if (!mbar_wait(&sfull_bar[slot], sph, abort_flag)) { ok = false; break; }
      const int tile = ring[slot * G_SLOT_INTS];
      TileInfo ti = slot_load(ring + slot * G_SLOT_INTS);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sempty_bar[slot]);
      if (tile < 0) break;
      const Segment& sg = p.seg[ti.seg];
      // this CTA's half of the 256-row tile
      ti.row0 += 128 * (int)rank;
      ti.rows = min(max(ti.rows - 128 * (int)rank, 0), 128);
      if (!__all_sync(0xffffffffu, mbar_wait(&tfull_bar[as], aphase, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + as * 256 + (static_cast<uint32_t>(q * 32) << 16);
      tc_epilogue<MODE>(p, ti, sg, taddr, stg, lane, q, 32);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (leader) mbar_arrive(&tempty_bar[as]);
        else mbar_arrive_cluster(tempty_leader[as]);
      }
      if (++as == 2) { as = 0; aphase ^= 1; }
    }
    if (!ok) { atomicCAS(p.status, 0, DEV_TIMEOUT); *abort_flag = 1; }
  }

  // ---------------------------------------------------------------- teardown
  // The next kernel of the stream may be scheduled from here on, not earlier: its CTAs then meet SMs that this
  // grid is about to leave, instead of sitting beside a pair whose tensor memory is still bound to two SMs.
  pdl_launch_dependents();
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies still in flight time to land before the shared memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  // Neither CTA may release its shared or tensor memory while the pair's MMAs, commits or remote arrivals can
  // still touch it: both meet here (every role has left its loop, by completion or by a run-out wait).
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_relinquish_pair();
    tmem_dealloc_pair(tmem_base, P_TMEM_COLS);
  }
  // the pair's tensor memory was allocated by both CTAs together and is given back by both together: neither
  // CTA leaves its SM before the other has issued its half of the de-allocation
  cluster_sync_all();
}

// ---------------------------------------------------------------- host side
fmmoe_status launch_ffn_tc2(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s) {
  const fmmoe_layer_desc& d = *a.d;
  const int H = d.hidden, I = d.inter, E = d.n_experts, Ns = d.n_shared, Is = d.shared_inter;
  if (!h->encode_tiled) return FMMOE_ERR_CUDA;
  if (a.T == 0) return FMMOE_OK;
  constexpr int BM2 = 2 * TC_BLOCK_M;
  const int mtps = (int)((a.T + BM2 - 1) / BM2);
  const uint64_t p_rows = (uint64_t)a.p_max;

  CUtensorMap A1r, A1s, G1r, U1r, G1s, U1s, A2r, A2s, D2r, D2s;
  bool ok = true;
  ok &= make_map(h, &A1r, a.xp, p_rows, H, 128);
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
    A1s = A1r; G1s = G1r; U1s = U1r; A2s = A2r; D2s = D2r;   // never dereferenced without shared experts
  }
  if (!ok) return FMMOE_ERR_CUDA;

  GemmParams p1 = {};
  p1.mtiles = a.mtiles; p1.n_mtiles = a.n_mtiles; p1.max_mtiles = a.max_mtiles;
  p1.block_m = BM2; p1.shared_mtiles = Ns * mtps; p1.mt_per_shared = mtps; p1.T = a.T;
  p1.seg[0] = Segment{(I + 127) / 128, H / P_BK, I, I, 0, 0, I};
  p1.seg[1] = Segment{Ns ? (Is + 127) / 128 : 0, H / P_BK, Is, Is, 0, (int)a.T, Is};
  p1.act[0] = static_cast<__nv_bfloat16*>(a.act); p1.act[1] = static_cast<__nv_bfloat16*>(a.act_sh);
  p1.status = a.d_status;
  p1.x = static_cast<const __nv_bfloat16*>(a.x); p1.ld_x = H; p1.row_token = a.row_token; p1.gather = 0;
  p1.tile_counter = a.tile_counters;
  p1.wait_budget_ns = h->wait_budget_ns; p1.test_withhold_stage = -1;

  GemmParams p2 = p1;
  p2.seg[0] = Segment{(H + 255) / 256, I / P_BK, H, H, 0, 0, H};
  p2.seg[1] = Segment{Ns ? (H + 255) / 256 : 0, Ns ? Is / P_BK : 0, H, H, (int)a.T, (int)a.T, H};
  p2.row_token = a.row_token; p2.row_gate = a.row_gate; p2.acc = a.acc;
  p2.y[0] = a.y; p2.y[1] = a.ysh; p2.deterministic = a.deterministic;
  p2.yb[0] = static_cast<__nv_bfloat16*>(a.yb); p2.yb[1] = static_cast<__nv_bfloat16*>(a.ybsh); p2.pair = a.pair;
  p2.tile_counter = a.tile_counters + 1;

  if (!h->tc2_attr_set) {
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_tc2_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES));
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(ffn_tc2_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES));
    h->tc2_attr_set = true;
  }
  const int grid = h->sm_count & ~1;      // whole CTA pairs
  { ProfScope ps(h, FMMOE_KERNEL_GEMM1, s); FMMOE_CUDA_TRY(launch_ex(ffn_tc2_kernel<0>, dim3(grid), dim3(P_THREADS), P_SMEM_BYTES, s, 2, false, A1r, A1s, G1r, U1r, G1s, U1s, p1)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  { ProfScope ps(h, FMMOE_KERNEL_GEMM2, s); FMMOE_CUDA_TRY(launch_ex(ffn_tc2_kernel<1>, dim3(grid), dim3(P_THREADS), P_SMEM_BYTES, s, 2, false, A2r, A2s, D2r, D2r, D2s, D2s, p2)); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 2;
  return FMMOE_OK;
}

}  // namespace fmmoe
