#define PLT_INST_D 64
#define PLT_INST_NT 3
#define PLT_INST_RW 2
#define PLT_INST_NAME main_bf16_d64_n3r2
#include "plt_main_bf16_inst.inl"
