#define PLT_INST_D 128
#define PLT_INST_MT 4
#define PLT_INST_NAME main_bf16_d128_mt4
#include "plt_main_bf16_inst.inl"
