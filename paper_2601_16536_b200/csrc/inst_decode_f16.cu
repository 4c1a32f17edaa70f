#define W4A16_INST_BF false
#define W4A16_INST_NAME f16
#include "inst_decode.cuh"
