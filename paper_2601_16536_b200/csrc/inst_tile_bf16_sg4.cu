#define W4A16_INST_BF true
#define W4A16_INST_SG 4
#define W4A16_INST_NAME bf16_sg4
#include "inst_tile.cuh"
