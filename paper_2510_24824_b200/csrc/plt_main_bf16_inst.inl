// Instantiates the bf16 main kernel for one (head dim, row tiles) pair and the (KV heads per block,
// key slices) variants that fit 8 consumer warps. Included by the plt_main_bf16_d*_mt*.cu files,
// which define PLT_INST_D, PLT_INST_MT and PLT_INST_NAME.
#include "plt_host.h"
#include "plt_main_bf16.cuh"

namespace plt {

namespace {

template <int HPC, int KW>
cudaError_t run_op(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t stream,
                   int* out) {
    constexpr int D = PLT_INST_D, MT = PLT_INST_MT;
    using C = MainCfg<D, MT, HPC, KW>;
    auto fn = plt_decode_main_bf16<D, MT, HPC, KW>;
    if (op == 0) return cudaSuccess;
    if (op == 1) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)v.smem);
        if (e != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, fn, C::NTHREADS, v.smem);
    }
    if (op == 3) {
        *out = (int)C::smem_bytes(v.stages, v.grid /* max_batch passed in grid for this query */);
        return cudaSuccess;
    }
    fn<<<v.grid, C::NTHREADS, v.smem, stream>>>(maps[0], maps[1], maps[2], maps[3], *p, v.stages);
    return cudaGetLastError();
}

}  // namespace

cudaError_t PLT_INST_NAME(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t stream,
                          int* out) {
#define PLT_CASE(H, K)                                               \
    if (v.HPC == H && v.KW == K) {                                   \
        if constexpr (H * K * PLT_INST_MT <= 8) return run_op<H, K>(op, v, maps, p, stream, out); \
    }
    PLT_CASE(1, 1) PLT_CASE(1, 2) PLT_CASE(1, 4) PLT_CASE(2, 1) PLT_CASE(2, 2) PLT_CASE(2, 4)
    PLT_CASE(4, 1) PLT_CASE(4, 2) PLT_CASE(8, 1)
#undef PLT_CASE
    return cudaErrorInvalidValue;
}

}  // namespace plt
