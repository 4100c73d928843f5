// Instantiations and launcher of the resident multi-step kernel.
#include "ds_resident_kernel.cuh"

namespace ds {

template <int CODE, int NOISE, int MAXT>
static cudaError_t launch_resident_one(const ResidentParams& rp, int num_sms, cudaStream_t stream) {
    auto kern = ds_resident_kernel<CODE, NOISE, MAXT>;
    const StepParams& p = rp.p;
    const size_t smem = resident_smem_layout(p.n, p.nnz).total;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)p.tiles), block((unsigned)p.n * 32u);
    if (!p.prescaled) {
        // per-chunk scales: blocks never wait for one another
        kern<<<grid, block, smem, stream>>>(rp);
        return cudaGetLastError();
    }
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, (int)block.x, smem);
    if (e != cudaSuccess) return e;
    if ((int64_t)per_sm * num_sms < p.tiles) return cudaErrorCooperativeLaunchTooLarge;
    e = cudaMemsetAsync(rp.barrier, 0, sizeof(unsigned int), stream);
    if (e != cudaSuccess) return e;
    void* args[] = {const_cast<ResidentParams*>(&rp)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kern), grid, block, args, smem, stream);
}

template <int CODE>
static cudaError_t launch_resident_code(int noise, const ResidentParams& rp, int num_sms, cudaStream_t stream) {
    const bool small = rp.p.n <= 4;
#define DS_RES_CASE(NZ) \
    if (noise == NZ) return small ? launch_resident_one<CODE, NZ, 128>(rp, num_sms, stream) \
                                  : launch_resident_one<CODE, NZ, 512>(rp, num_sms, stream);
    DS_RES_CASE(NOISE_NONE) DS_RES_CASE(NOISE_GAUSS) DS_RES_CASE(NOISE_T3)
#undef DS_RES_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_resident(int code, int noise, const ResidentParams& rp, int num_sms, cudaStream_t stream) {
    switch (code) {
        case CODE_SIGN: return launch_resident_code<CODE_SIGN>(noise, rp, num_sms, stream);
        case CODE_U2: return launch_resident_code<CODE_U2>(noise, rp, num_sms, stream);
        case CODE_U4: return launch_resident_code<CODE_U4>(noise, rp, num_sms, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ds
