// Parameters of the tcgen05 weight-streaming kernels (z2z_stream.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "z2z_common.cuh"
#include "z2z_internal.h"

namespace z2z {

constexpr int kMaxStages = 8;
constexpr int kGemmNT = 128;                    // weight rows per tile of the stream-K GEMM
constexpr int kLogitNT = 128, kLogitKSB = 1;
constexpr int kLogitGran = 32;                  // scheduling granule of the logits kernel, in weight rows (TMA boxes of
                                                // fewer rows stream several times slower)
constexpr int kLogitBoxClasses = 3;             // TMA boxes of 32, 64 and 128 weight rows

// Tensor maps of the logits kernel: hidden rows, then W_U and U_h once per box size.
struct LogitMaps {
  CUtensorMap h;
  CUtensorMap w[2 * kLogitBoxClasses];
};

// ---- decode logits kernel (z2z_decode_logits.cu) ---------------------------------------------
// Tensor maps, all of the form [k-block][row][64 columns]: hidden rows as one resident operand
// (h) and per stage with 1, 2 or 4 k-blocks (hk[0..2]); W_U and U_h as boxes of 64 rows x 2
// k-blocks (class 1) and 128 rows x 1 k-block (class 2): w[tensor * 2 + (class == 2)].
struct DecodeLogitMaps {
  CUtensorMap h, hk[3];
  CUtensorMap w[4];
};
struct DecodeLogitsParams {
  CbView cb;
  LogitsArgs la;
  int ksteps;            // d / 64 (a multiple of 4)
  int hid_rows;          // hidden rows held per k-block in shared memory (N rounded up to 8)
  int hid_box_kb;        // k-blocks per TMA box of the resident hidden rows
  int stages;            // stages of the load ring
  int part_stride;       // partial slots per hidden row
  int fixed_granules;    // 64-row granules of W_U every CTA owns up front
  int* counters;         // device words: [0] pool claims, [1] CTAs finished (both return to 0)
  int* err;
};
bool make_tmap_bf16_kblocks(CUtensorMap* m, const void* base, long long rows, long long cols, int box_rows,
                            int box_kb);
bool decode_logits_applies(const LogitsArgs& a);
cudaError_t run_logits_decode(const CbView& cb, const LogitsArgs& a, int* counters, int* err_word,
                              LogitsPartInfo* info, Prof* prof, cudaStream_t s);

// Stream-K GEMM over `groups` independent problems of identical shape (the two hyper-encoders).
// The unit space is (row tile, group, weight tile, k-step); CTA c of G owns units
// [floor(cU/G), floor((c+1)U/G)).  Every maximal run of units inside one tile and one CTA is one
// accumulator.  Operands are swapped with respect to the result's orientation: the 128 weight rows
// of a tile are the MMA's M, the activation rows its N, and a thread of the epilogue owns one
// output feature.
//
// The activation operand holds the hi part and the lo part of PACKED row r in rows 2r and 2r + 1
// (bf16 [2 * Rt, K]); only the first *rows_dev packed rows carry data, a count that only the device
// knows.  One TMA box of a_box_rows (= 2 * min(Rt, 128)) operand rows is loaded per stage; with a
// single row tile the MMA's N is 2 * P8 (P8 = live rows rounded up to 8): the tensor-core work
// and the epilogue's reductions follow the number of rows that exist, not the capacity of the
// pass.  The epilogue adds the hi and lo columns of a row in registers and reduces the sums into
// the fp32 result matrix out[group][Rt][J] (lanes = consecutive features = consecutive addresses).
struct StreamGemmParams {
  int row_tiles;         // 128-row tiles of the packed activation rows (outermost dimension of the unit space)
  int groups, tiles_per_group, ksteps;
  int ksb;               // 64-column k-blocks per stage and TMA box: 2 when the stages stay small, else 1
  int a_box_rows;        // operand rows per TMA box (multiple of 16, <= 256): the MMA's largest N
  float* out;            // [groups][Rt][J] fp32, zero before the first add
  int J, Rt;
  const int* rows_dev;   // device word: packed rows that carry data (<= Rt)
  int* err;
};

struct StreamLogitsParams {
  CbView cb;
  LogitsArgs la;
  int ksteps;
  int a_box_rows;
  int row_tiles;         // ceil(N / 128)
  int part_stride;       // partial slots per row
  int* vt_out;           // device word: number of virtual column tiles
  int* err;
};

// Prompt-scoring logits kernel (z2z_prefill_logits.cu): CTA pairs, 256 x 256 tiles.
constexpr int kPrefillMaxStrips = 8;            // column strips a row tile may be cut into
struct PrefillLogitsParams {
  CbView cb;
  LogitsArgs la;
  int ksteps;            // d / 64
  int row_tiles;         // ceil(N / 256)
  int n_static;          // ceil(V / 256)
  int strips;            // column strips per row tile = partial reductions per hidden row
  int32_t* tile_lo;      // [row_tiles] lowest / highest sequence owning a row of the tile
  int32_t* tile_hi;
  int32_t* tile_nh;      // [row_tiles] hypertoken column tiles of the tile
  int* err;
};

// CTA-pair GEMM of the prompt-sized hyper-encoder passes (z2z_pair_gemm.cu).
enum { kEpiStore = 0, kEpiResid = 1, kEpiGelu = 2 };
struct PairGemmParams {
  CbView cb;
  EntryList el;
  int R, Rt;             // row capacity of the pass; rows per hi (or lo) block of the operands
  const int* live_rows;  // device word: packed rows that carry data (rows of live entries, no padding)
  int J;                 // output columns (a multiple of 128)
  const void* bias;      // [J] bf16
  float* out;            // kEpiStore / kEpiResid: fp32 [R, J]
  __nv_bfloat16* out_hl; // kEpiGelu: bf16 [2 Rt, J], hi rows then lo rows (single fp16 operand: fp16 [Rt, J])
  int ksteps, row_tiles, col_tiles;
  int* err;
};
cudaError_t launch_pair_gemm(const PairGemmParams& p, const void* act, const void* W, int K, int epi, bool half,
                             cudaStream_t s);

bool make_tmap_bf16(CUtensorMap* m, const void* base, long long rows, long long cols, int box_rows);
int stream_gemm_stages(int ksb, int a_box_rows);
cudaError_t launch_stream_gemm(const StreamGemmParams& p, const CUtensorMap* maps, int grid, cudaStream_t s);
cudaError_t launch_stream_logits(const StreamLogitsParams& p, const LogitMaps* maps, int grid, bool merge,
                                 Prof* prof, cudaStream_t s);

}  // namespace z2z
