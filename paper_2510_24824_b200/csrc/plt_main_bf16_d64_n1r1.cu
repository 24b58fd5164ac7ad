#define PLT_INST_D 64
#define PLT_INST_NT 1
#define PLT_INST_RW 1
#define PLT_INST_NAME main_bf16_d64_n1r1
#include "plt_main_bf16_inst.inl"
