// Parameters shared by the two forms of the attention core (dsn_attention.cu, dsn_attention_ws.cu).
#pragma once

#include "dsn_internal.cuh"

constexpr int kAttTableGroups = 64;  // groups the persistent forms hold in their shared-memory item table

struct AttParams {
  CUtensorMap map;        // qkv seen as [sample][N rows][3H][64], box 1 x 128 rows x 1 x 64: rows >= N read as zeros
  CUtensorMap map_out;    // out seen as [sample][N rows][H * 64], box 1 x 32 rows x 64 columns (128-byte swizzle)
  int8_t heads[DSN_MAX_SLICES];
  int32_t N, H, B, G, T;
  int32_t grouped;        // 1: position p holds its data at row block p; 0: at row block perm[p]
  const int32_t* offsets;
  const int32_t* perm;
  const int32_t* group_slice;
  const __nv_bfloat16* qkv;
  int64_t ld_qkv;
  __nv_bfloat16* out;
  int64_t ld_out;
  int32_t* status;
};

// warp-specialised form: one persistent CTA per SM, item = (sample, head); needs G <= kAttTableGroups
size_t dsn_attention_ws_smem_bytes();
cudaError_t dsn_launch_attention_ws(const AttParams& p, int sm_count, cudaStream_t s);
