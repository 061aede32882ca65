// Layout of the tensor-core GEMM's activation operand in global memory.
//
// The operand A[M][K] (M activation rows, K a multiple of 64) is stored as the GEMM's shared-memory
// stages want it, so that a stage's activation part arrives with one contiguous bulk copy (no tensor map,
// one instruction per stage whatever the number of rows) instead of tiled TMA loads of 128-byte rows.
// Every SM re-reads the whole operand for each weight tile, so it stays in the L2; measured, the bytes
// an SM takes in per second (weights + activations together, about 75 GB/s) are the same either way.
//
//   [row chunk c][K block kb][part: 0 = bf16 high part, 1 = bf16 remainder][row r < NB][64 elements]
//
// with the 128-byte swizzle of the UMMA's K-major layout applied inside each row: the 16-byte piece
// p of row r sits at piece position p ^ (r mod 8).  Row chunks are NB = (M / chunks) rounded up to 16
// rows, chunks = ceil(M / 128).  Rows r >= the chunk's real row count are never read back.
#pragma once
#include <stdint.h>

struct OperandLayout {
  int NB;        // rows per chunk (multiple of 16, <= 128)
  int n_chunks;  // row chunks
  int n_kb;      // K / 64
};

inline OperandLayout operand_layout(int M, int K) {
  OperandLayout L;
  L.n_chunks = (M + 127) / 128;
  L.NB = ((M + L.n_chunks - 1) / L.n_chunks + 15) / 16 * 16;
  L.n_kb = K / 64;
  return L;
}
// elements of an operand buffer for M rows of K elements (both parts)
inline int64_t operand_elems(int M, int K) {
  const OperandLayout L = operand_layout(M, K);
  return (int64_t)L.n_chunks * L.n_kb * 2 * L.NB * 64;
}

#ifdef __CUDACC__
// element offset of (row m, column k, part) -- k's 8-element piece stays contiguous
__device__ __forceinline__ size_t operand_index(const OperandLayout& L, int m, int k, int part) {
  const int c = m / L.NB, r = m - c * L.NB;
  const int kb = k >> 6, kk = k & 63;
  return ((((size_t)c * L.n_kb + kb) * 2 + part) * L.NB + r) * 64 + ((((kk >> 3) ^ (r & 7)) << 3) | (kk & 7));
}
#endif
