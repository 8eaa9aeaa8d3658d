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
constexpr int G_EPI_LD = 33;                                 // padded row of the epilogue transpose buffer
constexpr int G_EPI_BYTES = 4 * 32 * G_EPI_LD * 4;           // one 32x32 fp32 block per epilogue warp

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
  int block_m;                // rows per M-tile of the tile list (128; 256 for CTA pairs)
  int shared_mtiles;          // N_s * ceil(T/block_m), host-known
  int mt_per_shared;          // ceil(T/block_m)
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
    ti.row0 = mb * p.block_m;
    const long long left = p.T - (long long)ti.row0;
    ti.rows = left < p.block_m ? (int)left : p.block_m;
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

// Epilogue of one tile for one epilogue warp: the warp owns TMEM lane quarter q (taddr already points at it and
// at the accumulator stage), i.e. `rpw` rows of the tile starting at tile row q * rpw (32 rows, or 16 when a tile
// of at most 64 rows ran as M = 64 MMAs).  `ti` describes the 128-row tile this CTA holds.  `stg` is the warp's
// 32 x 33 fp32 staging block.
//   MODE 0: SwiGLU of the gate / up columns -> act (bf16), coalesced through the staging block.
//   MODE 1: gate scaling, then per-pair bf16 rows (pair-row mode), fp32 rows (fixed-order mode) or vector
//           reductions into the fp32 accumulator.
template <int MODE>
__device__ __forceinline__ void tc_epilogue(const GemmParams& p, const TileInfo& ti, const Segment& sg, uint32_t taddr,
                                            float* stg, int lane, int q, int rpw) {
  const int rows_w = min(ti.rows - q * rpw, rpw);   // valid rows among this warp's (may be <= 0)
  const long long out_row0 = (long long)ti.row0 + q * rpw + (long long)ti.group_local * sg.out_group_stride;
  const int r = q * rpw + lane;                     // row of the tile held by this thread (if lane < rpw)
  if (MODE == 0) {
    uint32_t* stg32 = reinterpret_cast<uint32_t*>(stg);   // [32][17] packed bf16 pairs
    __nv_bfloat16* dst0 = p.act[ti.seg] + out_row0 * sg.ld_out + ti.nb * 128;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      if (ti.nb * 128 + c * 32 >= sg.n_valid) break;   // warp-uniform
      uint32_t g[32], u[32];
      tmem_ld32(taddr + c * 32, g);
      tmem_ld32(taddr + 128 + c * 32, u);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
        const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(u[2 * i]);
        const float a1 = __fdividef(g1, 1.f + __expf(-g1)) * __uint_as_float(u[2 * i + 1]);
        const __nv_bfloat162 h = __floats2bfloat162_rn(a0, a1);
        stg32[lane * 17 + i] = *reinterpret_cast<const uint32_t*>(&h);
      }
      __syncwarp();
      // 4 lanes x 16 bytes cover the 64-byte row segment; 8 rows per instruction
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const int row = rr * 8 + (lane >> 2);
        const int w4 = (lane & 3) * 4;
        if (row < rows_w) {
          const uint32_t* sp = stg32 + row * 17 + w4;
          *reinterpret_cast<uint4*>(dst0 + (long long)row * sg.ld_out + c * 32 + w4 * 2) =
              make_uint4(sp[0], sp[1], sp[2], sp[3]);
        }
      }
      __syncwarp();
    }
  } else {
    int tok; float gate;
    if (ti.seg == 0) {
      const bool row_ok = lane < rows_w;
      tok = row_ok ? p.row_token[ti.row0 + r] : 0;
      gate = row_ok ? p.row_gate[ti.row0 + r] : 0.f;
    } else {
      tok = ti.row0 + r; gate = 1.f;
    }
    if (p.deterministic) gate = 1.f;   // gates are applied by the ordered gather
    float* ybase = p.deterministic ? p.y[ti.seg] + out_row0 * sg.ld_out + ti.nb * 256 : nullptr;
    if (p.pair) {
      // Pair-row mode: gate-scaled bf16 rows per pair.  As in GEMM-1's epilogue the 32 x 32 block goes through
      // the staging block so that every store instruction writes whole 64-byte row segments (4 lanes x 16
      // bytes per row, 8 rows per instruction) instead of 32 quarter-segments of 32 different rows.
      uint32_t* stg32 = reinterpret_cast<uint32_t*>(stg);   // [32][17] packed bf16 pairs
      __nv_bfloat16* y0 = p.yb[ti.seg] + out_row0 * sg.ld_out + ti.nb * 256;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        if (ti.nb * 256 + c * 32 >= sg.n_valid) break;   // warp-uniform
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const __nv_bfloat162 hh = __floats2bfloat162_rn(gate * __uint_as_float(v[2 * i]), gate * __uint_as_float(v[2 * i + 1]));
          stg32[lane * 17 + i] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        __syncwarp();
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
          const int row = rr * 8 + (lane >> 2);
          const int w4 = (lane & 3) * 4;
          if (row < rows_w) {
            const uint32_t* sp = stg32 + row * 17 + w4;
            *reinterpret_cast<uint4*>(y0 + (long long)row * sg.ld_out + c * 32 + w4 * 2) = make_uint4(sp[0], sp[1], sp[2], sp[3]);
          }
        }
        __syncwarp();
      }
    } else
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      if (ti.nb * 256 + c * 32 >= sg.n_valid) break;   // warp-uniform
      uint32_t v[32];
      tmem_ld32(taddr + c * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) stg[lane * G_EPI_LD + j] = gate * __uint_as_float(v[j]);
      __syncwarp();
      // 8 lanes x 16 bytes cover a row's 128-byte segment; 4 rows per instruction
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        const int row = rr * 4 + (lane >> 3);
        const int col = (lane & 7) * 4;
        const int tok_r = __shfl_sync(0xffffffffu, tok, row);
        if (row < rows_w) {
          const float* sp = stg + row * G_EPI_LD + col;
          if (p.deterministic) {
            *reinterpret_cast<float4*>(ybase + (long long)row * sg.ld_out + c * 32 + col) =
                make_float4(sp[0], sp[1], sp[2], sp[3]);
          } else {
            red_add_v4(p.acc + (long long)tok_r * sg.ld_out + ti.nb * 256 + c * 32 + col, sp[0], sp[1], sp[2], sp[3]);
          }
        }
      }
      __syncwarp();
    }
  }
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
