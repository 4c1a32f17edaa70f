// The GEMM kernels are compiled in several translation units (one per 16-bit type and group size); each
// unit hands out its instantiations through the functions below and owns one device status word.
#pragma once

#include "kernel_decode.cuh"
#include "kernel_tile.cuh"

namespace w4a16 {

typedef void (*DecodeKernel)(const CUtensorMap, const DecodeParams);
typedef void (*TileKernel)(const CUtensorMap, const TileParams);

// sg = scale rows per 128-k block (1, 2, 4)
// a_box: activation rows of a stage as one tensor copy
DecodeKernel decode_kernel_f16(int mb, bool cluster, int sg, bool sym, bool a_box);
DecodeKernel decode_kernel_bf16(int mb, bool cluster, int sg, bool sym, bool a_box);
TileKernel tile_kernel_f16_sg1(int mt_index, bool sym, bool epi);
TileKernel tile_kernel_f16_sg2(int mt_index, bool sym, bool epi);
TileKernel tile_kernel_f16_sg4(int mt_index, bool sym, bool epi);
TileKernel tile_kernel_bf16_sg1(int mt_index, bool sym, bool epi);
TileKernel tile_kernel_bf16_sg2(int mt_index, bool sym, bool epi);
TileKernel tile_kernel_bf16_sg4(int mt_index, bool sym, bool epi);

int status_take_decode_f16();
int status_take_decode_bf16();
int status_take_tile_f16_sg1();
int status_take_tile_f16_sg2();
int status_take_tile_f16_sg4();
int status_take_tile_bf16_sg1();
int status_take_tile_bf16_sg2();
int status_take_tile_bf16_sg4();

}  // namespace w4a16
