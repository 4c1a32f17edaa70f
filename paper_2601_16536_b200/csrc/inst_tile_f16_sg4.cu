#define W4A16_INST_BF false
#define W4A16_INST_SG 4
#define W4A16_INST_NAME f16_sg4
#include "inst_tile.cuh"
