// Instantiates the branch-fused kernels for one held-operand width (compile with -DMPQ_HB=1..8):
// eight translation units build in parallel and together cover all 64 (a_bits, w_bits) pairs.
#include "mpq_branch_launch.cuh"
#include "mpq_pointwise_kernel.cuh"

#ifndef MPQ_HB
#error "compile with -DMPQ_HB=<1..8>"
#endif

namespace mpq {

template <>
int launch_gemm_hb<MPQ_HB>(int sb, const BranchParams& p, cudaStream_t st) {
    switch (sb) {
        case 1: return launch_auto<MPQ_HB, 1, kModeGemm>(p, st);
        case 2: return launch_auto<MPQ_HB, 2, kModeGemm>(p, st);
        case 3: return launch_auto<MPQ_HB, 3, kModeGemm>(p, st);
        case 4: return launch_auto<MPQ_HB, 4, kModeGemm>(p, st);
        case 5: return launch_auto<MPQ_HB, 5, kModeGemm>(p, st);
        case 6: return launch_auto<MPQ_HB, 6, kModeGemm>(p, st);
        case 7: return launch_auto<MPQ_HB, 7, kModeGemm>(p, st);
        case 8: return launch_auto<MPQ_HB, 8, kModeGemm>(p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

template <>
int launch_conv_hb<MPQ_HB>(int sb, const BranchParams& p, cudaStream_t st) {
    switch (sb) {
        case 1: return launch_auto<MPQ_HB, 1, kModeConv>(p, st);
        case 2: return launch_auto<MPQ_HB, 2, kModeConv>(p, st);
        case 3: return launch_auto<MPQ_HB, 3, kModeConv>(p, st);
        case 4: return launch_auto<MPQ_HB, 4, kModeConv>(p, st);
        case 5: return launch_auto<MPQ_HB, 5, kModeConv>(p, st);
        case 6: return launch_auto<MPQ_HB, 6, kModeConv>(p, st);
        case 7: return launch_auto<MPQ_HB, 7, kModeConv>(p, st);
        case 8: return launch_auto<MPQ_HB, 8, kModeConv>(p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

template <>
int launch_pointwise_hb<MPQ_HB>(int sb, const BranchParams& p, cudaStream_t st) {
    switch (sb) {
        case 1: return launch_pointwise<MPQ_HB, 1>(p, st);
        case 2: return launch_pointwise<MPQ_HB, 2>(p, st);
        case 3: return launch_pointwise<MPQ_HB, 3>(p, st);
        case 4: return launch_pointwise<MPQ_HB, 4>(p, st);
        case 5: return launch_pointwise<MPQ_HB, 5>(p, st);
        case 6: return launch_pointwise<MPQ_HB, 6>(p, st);
        case 7: return launch_pointwise<MPQ_HB, 7>(p, st);
        case 8: return launch_pointwise<MPQ_HB, 8>(p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

template <>
int launch_window3x3c64_hb<MPQ_HB>(int sb, const BranchParams& p, cudaStream_t st) {
    switch (sb) {
        case 1: return launch_window3x3c64<MPQ_HB, 1>(p, st);
        case 2: return launch_window3x3c64<MPQ_HB, 2>(p, st);
        case 3: return launch_window3x3c64<MPQ_HB, 3>(p, st);
        case 4: return launch_window3x3c64<MPQ_HB, 4>(p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

}  // namespace mpq
