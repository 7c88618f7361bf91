// The warp-level tensor-core instruction m16n8k16 (FP32 accumulation of exact 16-bit products), for the thin products
// that are not worth the tensor-memory path.  Fragment layout, with grp = lane / 4 and tig = lane % 4:
//   A (16 x 16, row-major): a0 = (row grp, cols 2 tig, 2 tig + 1), a1 = (row grp + 8, same cols),
//                           a2 = (row grp, cols 2 tig + 8, + 9),   a3 = (row grp + 8, those cols);
//   B (16 x 8, column-major): b0 = (rows 2 tig, 2 tig + 1 of column grp), b1 = (rows 2 tig + 8, + 9 of it);
//   C (16 x 8): c0, c1 = (row grp, cols 2 tig, 2 tig + 1), c2, c3 = (row grp + 8, those cols).
// A sum over k does not care in which order k is walked: a thread that feeds the 32-bit words of one contiguous
// quarter of its row, in pairs, as (a0, a2) or (b0, b1) of successive k-steps presents the same permutation of k on
// both sides as long as both operands are cut the same way.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace ahakv {

template <typename T> struct Mma16816;
template <> struct Mma16816<__half> {
  static __device__ __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
};
template <> struct Mma16816<__nv_bfloat16> {
  static __device__ __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
};

}  // namespace ahakv
