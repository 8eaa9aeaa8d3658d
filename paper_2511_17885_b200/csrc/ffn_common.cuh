// Pieces shared by the two forms of the grouped expert GEMM (ffn_tc.cu: token rows as the MMA's M
// dimension; ffn_sm.cu: token rows as its N dimension): the tile list arithmetic, the decoded-tile ring
// slot, and the tensor-map helper.
#pragma once
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int G_SCHED = 4;         // slots of the tile ring
constexpr int G_SLOT_INTS = 8;     // a slot: tile id (-1: no more tiles) + the decoded TileInfo

struct Segment {          // routed experts (0) or shared experts (1)
  int n_nblocks;          // N-blocks per group
  int k_blocks;           // K / 64
  int b_rows_per_group;   // rows of the B tensor per group (S_m for GEMM-1, H for GEMM-2)
  int n_valid;            // valid output columns per group (S_m for GEMM-1, H for GEMM-2)
  int a_group_stride;     // rows added to the A row per group index (shared experts only)
  int out_group_stride;   // rows added to the output row per group index
  int ld_out;             // leading dimension of the output (elements)
};

struct GemmParams {
  const MTile* mtiles;        // routed M-tiles
  const int32_t* n_mtiles;    // device: number of routed M-tiles
  int max_mtiles;             // capacity of `mtiles` (a corrupt count must not walk past it)
  int32_t* tile_counter;      // device: next tile to hand out (zero at launch)
  int shared_mtiles;          // N_s * ceil(T/128), host-known
  int mt_per_shared;          // ceil(T/128)
  long long T;
  Segment seg[2];
  // epilogue
  __nv_bfloat16* act[2];      // MODE 0: activation outputs (routed, shared)
  const __nv_bfloat16* x; int ld_x;   // MODE 0: hidden states [T, H] the routed rows are gathered from
  const int32_t* row_token;   // grouped row -> token (MODE 0: gather, MODE 1: combine)
  const float* row_gate;      // MODE 1
  float* acc;                 // MODE 1 atomic:  [T, H]
  float* y[2];                // MODE 1 deterministic: routed [P, H], shared [N_s*T, H]
  __nv_bfloat16* yb[2];       // MODE 1 pair-row mode: gate-scaled outputs per pair, bf16, same shapes
  int deterministic;
  int pair;                   // MODE 1: write yb instead of reducing into acc
  int gather;                 // MODE 0: routed rows come from x through the loader warps (else from the tmA_r map)
  int* status;
  const int8_t* wscale[2][2];          // FP8 weight stream: block scale exponents, [segment][weight box of the stage]
  unsigned long long wait_budget_ns;   // time budget of every bounded wait (ffn_sm.cu)
  int test_withhold_stage;             // self-test: the producer stops before this k-block (-1: never)
};

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

struct TileInfo {
  int seg, group_local, row0, rows, nb;
  bool single;   // routed: the expert's rows fit this one M-tile
};

// Position `tile` of the interleaved order -> (segment, M-tile, N-block).
__device__ __forceinline__ TileInfo decode_tile(const GemmParams& p, int tile, int n_mt_r) {
  TileInfo ti;
  const unsigned long long R = (unsigned long long)n_mt_r * p.seg[0].n_nblocks;
  const unsigned long long S = (unsigned long long)p.shared_mtiles * p.seg[1].n_nblocks;
  const unsigned long long N = R + S;
  const unsigned long long sb = (unsigned long long)tile * S / N;          // shared tiles before this position
  const unsigned long long sb1 = (unsigned long long)(tile + 1) * S / N;
  if (sb1 == sb) {
    const int r = tile - (int)sb;
    const int mt = r / p.seg[0].n_nblocks;
    ti.seg = 0;
    ti.nb = r - mt * p.seg[0].n_nblocks;
    const MTile m = p.mtiles[mt];
    ti.group_local = m.group; ti.row0 = m.row0; ti.rows = m.rows;
    ti.single = m.pad != 0;
  } else {
    const int t2 = (int)sb;
    ti.seg = 1;
    ti.nb = t2 / p.shared_mtiles;
    const int mt = t2 - ti.nb * p.shared_mtiles;
    ti.group_local = mt / p.mt_per_shared;
    const int mb = mt - ti.group_local * p.mt_per_shared;
    ti.row0 = mb * TC_BLOCK_M;
    const long long left = p.T - (long long)ti.row0;
    ti.rows = left < TC_BLOCK_M ? (int)left : TC_BLOCK_M;
    ti.single = false;
  }
  return ti;
}

// A slot of the tile ring as the producer publishes it and the other roles read it.
__device__ __forceinline__ void slot_store(volatile int* s, int tile, const TileInfo& ti) {
  s[0] = tile; s[1] = ti.seg; s[2] = ti.group_local; s[3] = ti.row0; s[4] = ti.rows; s[5] = ti.nb; s[6] = ti.single;
}
__device__ __forceinline__ TileInfo slot_load(const volatile int* s) {
  TileInfo ti;
  ti.seg = s[1]; ti.group_local = s[2]; ti.row0 = s[3]; ti.rows = s[4]; ti.nb = s[5]; ti.single = s[6] != 0;
  return ti;
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 row-major [rows, cols] tensor, box = 64 columns x box_rows rows, 128-byte swizzle.
static inline bool make_map(fmmoe_handle* h, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  if (rows == 0) rows = 1;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(h->encode_tiled)(
      m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}


// FP8 bytes, row-major [rows, cols], box = 64 bytes x box_rows rows, no swizzle (read by threads, not by the MMA).
static inline bool make_map_u8(fmmoe_handle* h, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  if (rows == 0) rows = 1;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(h->encode_tiled)(
      m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace fmmoe
