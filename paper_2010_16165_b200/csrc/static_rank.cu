// fp_rank_filters_static: filter scoring + ranking + masking for one filter bank without any
// device allocation.  The only intermediate the two kernels need - one fp64 score per filter -
// lives in a fixed array that is part of the library image.
#include "../../include/fupruner.h"
#include "fp_internal.h"

#include <mutex>

namespace {

// Scratch shared by every call on a device: scores of up to FP_STATIC_RANK_MAX_FILTERS filters.
// Every GPU that loads the library holds these 32 KB until the process exits.
static __device__ __align__(256) double g_static_scores[FP_STATIC_RANK_MAX_FILTERS];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
double* g_scores_ptr[kMaxDevices] = {};   // device address of g_static_scores, per device ordinal

}  // namespace

extern "C" const char* fp_last_error(void);
namespace fp_detail { fp_status set_error(fp_status st, const char* msg); }

extern "C" fp_status fp_rank_filters_static(const float* d_filters, int32_t K, int32_t per_filter, int32_t norm,
                                            int32_t q, int32_t* d_rank, uint8_t* d_mask, void* stream) {
    if (!d_filters || !d_rank || !d_mask) return fp_detail::set_error(FP_ERR_ARG, "fp_rank_filters_static: NULL argument");
    if (K <= 0 || per_filter <= 0 || q < 0 || q > K) return fp_detail::set_error(FP_ERR_ARG, "fp_rank_filters_static: bad sizes");
    if (norm != FP_NORM_L1 && norm != FP_NORM_L2) return fp_detail::set_error(FP_ERR_ARG, "fp_rank_filters_static: bad norm");
    if (K > FP_STATIC_RANK_MAX_FILTERS)
        return fp_detail::set_error(FP_ERR_BOUNDS, "fp_rank_filters_static: more filters than the built-in scratch holds (max 4096)");
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fp_detail::set_error(FP_ERR_CUDA, "fp_rank_filters_static: cannot identify the current device");
    double* scores = nullptr;
    {
        // One-time set-up per device, with that device current: in host code the array's name is only a
        // handle; the address a kernel can use has to be asked for.
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scores_ptr[dev]) {
            double* p = nullptr;
            cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scores);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                return fp_detail::set_error(FP_ERR_CUDA, "fp_rank_filters_static: cudaGetSymbolAddress failed");
            }
            g_scores_ptr[dev] = p;
        }
        scores = g_scores_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    // Both kernels overwrite everything they later read (scores[0..K)), so nothing has to be cleared.
    fp::launch_score_filters(d_filters, K, per_filter, norm, scores, st);
    fp::launch_rank_mask(scores, K, q, d_rank, d_mask, st);
    if (cudaGetLastError() != cudaSuccess) return fp_detail::set_error(FP_ERR_CUDA, "fp_rank_filters_static: kernel launch failed");
    return FP_OK;
}
