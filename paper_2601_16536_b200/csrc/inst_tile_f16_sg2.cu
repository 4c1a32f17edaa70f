#define W4A16_INST_BF false
#define W4A16_INST_SG 2
#define W4A16_INST_NAME f16_sg2
#include "inst_tile.cuh"
