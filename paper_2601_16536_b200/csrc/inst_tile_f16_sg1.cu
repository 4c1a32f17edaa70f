#define W4A16_INST_BF false
#define W4A16_INST_SG 1
#define W4A16_INST_NAME f16_sg1
#include "inst_tile.cuh"
