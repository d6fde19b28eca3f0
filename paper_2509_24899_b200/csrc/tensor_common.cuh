// Pieces shared by the tensor-core kernels (Q pass, K pass, first feature-map layer): tile loads,
// UMMA shared-memory descriptors for the two operand layouts in use, the swizzled row store, and the host
// helper that encodes a tensor map.
#pragma once

#include <cuda.h>

#include "as_internal.h"
#include "sm100_ptx.cuh"
#include "sm100_tmem_wide.cuh"

namespace as_tc {

using namespace sm100;

constexpr int BOX_BYTES = 128 * 128;     // one TMA box: 128 rows x 64 bf16 (128 bytes per row)

// Loads `nboxes` swizzled boxes [128 rows x 64 columns] starting at column x0, row y0 of slice z.
AS_DEV void load_boxes(uint32_t dst, const CUtensorMap* m, uint32_t bar, int x0, int y0, int z, int nboxes) {
  for (int b = 0; b < nboxes; ++b) tma_load_3d(dst + b * BOX_BYTES, m, bar, x0 + b * 64, y0, z);
}
// Loads a [128 x D] tile (rows y0.., of slice z) as D/64 swizzled boxes.
template <int D>
AS_DEV void load_tile(uint32_t dst, const CUtensorMap* m, uint32_t bar, int y0, int z) {
#pragma unroll
  for (int b = 0; b < D / 64; ++b) tma_load_3d(dst + b * BOX_BYTES, m, bar, b * 64, y0, z);
}

// Shared-memory descriptors are built once per tile; the k-steps of one MMA chain only add a byte
// offset (in 16-byte units) to the address field, which keeps the issuing thread's instruction count low.
AS_DEV uint64_t kmajor_desc(uint32_t smem) { return make_sdesc(smem, 16, 1024); }        // [rows x 64] boxes, K-major
AS_DEV uint64_t mnmajor_desc(uint32_t smem) { return make_sdesc(smem, BOX_BYTES, 1024); } // k-rows x [64-column boxes], MN-major
// offset of k-step kk (16 elements) inside a K-major tile of 64-column boxes
AS_DEV constexpr uint64_t kstep_kmajor(int kk) { return (uint64_t)(((kk / 4) * BOX_BYTES + (kk % 4) * 32) >> 4); }
// offset of k-step kk (16 rows) inside an MN-major tile
AS_DEV constexpr uint64_t kstep_mnmajor(int kk) { return (uint64_t)((kk * 2048) >> 4); }

// D[tmem] (+)= A[smem, K-major, 128 x KD] * B[smem, K-major, NB x KD]^T
template <int KD>
AS_DEV void issue_kmajor(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool acc) {
#pragma unroll
  for (int kk = 0; kk < KD / 16; ++kk)
    mma_ss(d_tmem, a_desc + kstep_kmajor(kk), b_desc + kstep_kmajor(kk), idesc, (acc || kk > 0) ? 1u : 0u);
}
// D[tmem] (+)= A[tmem, 128 lanes x 128 k as packed bf16] * B[smem, MN-major: 128 k-rows x NB cols]
AS_DEV void issue_tmemA_mnB(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool acc) {
#pragma unroll
  for (int kk = 0; kk < 8; ++kk)
    mma_ts(d_tmem, a_tmem + kk * 8, b_desc + kstep_mnmajor(kk), idesc, (acc || kk > 0) ? 1u : 0u);
}

// Writes 32 consecutive columns [c0, c0+32) of row `row` of a swizzled [128 x D] bf16 tile (1024-byte aligned).
// Through a 32-bit shared-memory address and st.shared: run by itself, the Q pass's per-tile instruction stream
// takes an eighth longer with the same stores issued through the generic pointer.  The row's 16-byte chunk c
// sits at (row start + ((row & 7) << 4)) ^ (c << 4): one xor per store.
AS_DEV void store_row_chunk(uint8_t* tile, uint32_t row, uint32_t c0, const uint32_t (&w)[16]) {
  const uint32_t base = smem_u32(tile) + (c0 / 64) * BOX_BYTES + row * 128u + ((row & 7u) << 4);
  const uint32_t chunk0 = (c0 % 64) / 8;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(base ^ ((chunk0 + i) << 4)), "r"(w[4 * i]), "r"(w[4 * i + 1]), "r"(w[4 * i + 2]), "r"(w[4 * i + 3])
                 : "memory");
}

// 3-D bf16 tensor [slices][rows][cols] (cols contiguous) viewed through boxes of 64 cols x box_rows rows
// with the 128-byte swizzle.  False when the driver entry point is missing or rejects the arguments.
bool make_map(CUtensorMap* m, const void* base, int cols, int rows, int slices, int box_rows);

template <typename K>
cudaError_t opt_in_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

}  // namespace as_tc

// Per-device set-up of each translation unit's kernels (shared-memory opt-in).
cudaError_t as_tensor_init_qpass();
cudaError_t as_tensor_init_kpass();
cudaError_t as_tensor_init_qstream();
