// Tensor-core causal varlen GQA prefill attention (placeholder until the tcgen05 kernel lands).
#include "common.cuh"
namespace skv {
bool tc_attention_supported(int, int, int) { return false; }
int launch_attention_tc(const bf16 *, const bf16 *, const bf16 *, bf16 *, const int32_t *, int, int, int, int, int, int,
                        unsigned int *, cudaStream_t) { return SWIFTKV_ERR_UNSUPPORTED; }
}  // namespace skv
