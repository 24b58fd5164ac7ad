// Instantiates the bf16 main kernel for one (head dim, 8-row groups per warp, warps along the rows)
// triple and the (KV heads per block, warps along the keys, slices per warp) variants that fit 8
// consumer warps. Included by the plt_main_bf16_d*_n*r*.cu files, which define PLT_INST_D,
// PLT_INST_NT, PLT_INST_RW and PLT_INST_NAME; PLT_INST_FP8 (default 0) selects the kernel for caches of E4M3 codes,
// which is built for the variants with two slices per warp only.
#include "plt_host.h"
#include "plt_main_bf16.cuh"

#ifndef PLT_INST_FP8
#define PLT_INST_FP8 0
#endif

namespace plt {

namespace {

template <int HPC, int KW, int KS>
cudaError_t run_op(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t stream,
                   int* out) {
    constexpr int D = PLT_INST_D, NT = PLT_INST_NT, RW = PLT_INST_RW;
    constexpr bool FP8 = PLT_INST_FP8 != 0;
    using C = TCfg<D, NT, RW, HPC, KW, KS, FP8>;
    auto fn = plt_decode_main_bf16<D, NT, RW, HPC, KW, KS, FP8>;
    if (op == 0) return cudaSuccess;
    if (op == 1) {
        cudaError_t e = allow_max_dynamic_smem((const void*)fn);
        if (e != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, fn, C::NTHREADS, v.smem);
    }
    if (op == 4) {
        *out = C::TK;
        return cudaSuccess;
    }
    if (op == 3) {
        *out = (int)C::smem_bytes(v.stages, v.grid /* max_batch passed in grid for this query */);
        return cudaSuccess;
    }
    // op 2: plain launch; op 5: launch with programmatic stream serialisation (this grid's blocks are set up while the
    // kernel before it in the stream finishes and wait for its completion in grid_dependency_wait()).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)v.grid);
    cfg.blockDim = dim3(C::NTHREADS);
    cfg.dynamicSmemBytes = v.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = op == 5 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, fn, maps[0], maps[1], maps[2], maps[3], *p, v.stages);
}

}  // namespace

cudaError_t PLT_INST_NAME(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t stream,
                          int* out) {
#define PLT_CASE(H, K, S)                                            \
    if (v.HPC == H && v.KW == K && v.KS == S) {                      \
        if constexpr (H * K * PLT_INST_RW <= (PLT_INST_NT <= 2 ? 8 : 4) && (!PLT_INST_FP8 || S == 2)) \
            return run_op<H, K, S>(op, v, maps, p, stream, out);                              \
    }
    PLT_CASE(1, 1, 1) PLT_CASE(1, 2, 1) PLT_CASE(1, 4, 1) PLT_CASE(2, 1, 1) PLT_CASE(2, 2, 1) PLT_CASE(2, 4, 1)
    PLT_CASE(1, 8, 1) PLT_CASE(4, 1, 1) PLT_CASE(4, 2, 1) PLT_CASE(8, 1, 1)
    PLT_CASE(1, 1, 2) PLT_CASE(1, 2, 2) PLT_CASE(1, 4, 2) PLT_CASE(2, 1, 2) PLT_CASE(2, 2, 2) PLT_CASE(4, 1, 2)
#undef PLT_CASE
    return cudaErrorInvalidValue;
}

}  // namespace plt
