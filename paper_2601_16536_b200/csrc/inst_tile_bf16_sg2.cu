#define W4A16_INST_BF true
#define W4A16_INST_SG 2
#define W4A16_INST_NAME bf16_sg2
#include "inst_tile.cuh"
