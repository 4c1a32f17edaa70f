#define W4A16_INST_BF true
#define W4A16_INST_SG 1
#define W4A16_INST_NAME bf16_sg1
#include "inst_tile.cuh"
