// bf16 expert FFN dispatch (bring-up version: CUDA-core kernel for both classes).
#include "common.cuh"

namespace monde {

int launch_ffn_bf16(const monde_problem& p, const void* x_perm, const void* W1, const void* b1,
                    const void* W2, const void* b2, const int32_t* counts, const int32_t* offsets,
                    const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                    void* y_perm, void* ws, cudaStream_t s) {
    void* h = static_cast<char*>(ws) + WsLayout::kHidden;
    const int32_t* lists[2] = {hot_ids, cold_ids};
    for (int c = 0; c < 2; ++c) {
        int st = launch_linear_simt(p.dtype, p.act, p.E, p.d_model, p.d_ff, x_perm, W1, b1, offsets, lists[c],
                                    n_hot_cold + c, h, s);
        if (st != MONDE_OK) return st;
        st = launch_linear_simt(p.dtype, -1, p.E, p.d_ff, p.d_model, h, W2, b2, offsets, lists[c],
                                n_hot_cold + c, y_perm, s);
        if (st != MONDE_OK) return st;
    }
    return MONDE_OK;
}

}  // namespace monde
