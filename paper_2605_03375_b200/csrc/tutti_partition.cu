// SM partition for the capped mode: an "I/O control domain" of a few SMs and a
// "compute domain" with the rest, isolated with CUDA green contexts (paper Section
// 3.2, "SM Partitioning For Accurate I/O").  The driver entry points are looked up
// at run time so that the library itself does not link against libcuda.
#include <cuda.h>

#include <string>

#include "tutti_internal.h"

struct tutti_ctx;   // defined in tutti_lib.cu; only the accessors below touch it

namespace tutti {
struct PartitionState {
    CUgreenCtx io = nullptr, compute = nullptr;
    CUstream io_stream = nullptr, compute_stream = nullptr;
};
}  // namespace tutti

using namespace tutti;

extern "C" void **tutti_ctx_partition_slot_(tutti_ctx_t *ctx);   // storage for a PartitionState*
extern "C" int tutti_ctx_device_(tutti_ctx_t *ctx);
extern "C" void tutti_set_cuda_error_(const char *msg);

namespace {

template <typename F>
bool load(const char *name, F *fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || !p ||
        q != cudaDriverEntryPointSuccess)
        return false;
    *fn = reinterpret_cast<F>(p);
    return true;
}

int fail(const char *what, CUresult r) {
    std::string m = std::string(what) + ": CUresult " + std::to_string((int)r);
    tutti_set_cuda_error_(m.c_str());
    return TUTTI_ECUDA;
}

}  // namespace

extern "C" int tutti_sm_partition_create(tutti_ctx_t *ctx, uint32_t io_sms, void **io_stream,
                                         void **compute_stream, uint32_t *io_sms_got,
                                         uint32_t *compute_sms_got) {
    if (!ctx || !io_stream || !compute_stream || io_sms == 0) return TUTTI_EINVAL;
    void **slot = tutti_ctx_partition_slot_(ctx);
    if (*slot) return TUTTI_EINVAL;   // one partition per context
    CUresult (*pDeviceGet)(CUdevice *, int) = nullptr;
    CUresult (*pGetDevResource)(CUdevice, CUdevResource *, CUdevResourceType) = nullptr;
    CUresult (*pSplit)(CUdevResource *, unsigned int *, const CUdevResource *, CUdevResource *,
                       unsigned int, unsigned int) = nullptr;
    CUresult (*pGenDesc)(CUdevResourceDesc *, CUdevResource *, unsigned int) = nullptr;
    CUresult (*pGreenCreate)(CUgreenCtx *, CUdevResourceDesc, CUdevice, unsigned int) = nullptr;
    CUresult (*pGreenStream)(CUstream *, CUgreenCtx, unsigned int, int) = nullptr;
    CUresult (*pGreenDestroy)(CUgreenCtx) = nullptr;
    if (!load("cuDeviceGet", &pDeviceGet) || !load("cuDeviceGetDevResource", &pGetDevResource) ||
        !load("cuDevSmResourceSplitByCount", &pSplit) ||
        !load("cuDevResourceGenerateDesc", &pGenDesc) || !load("cuGreenCtxCreate", &pGreenCreate) ||
        !load("cuGreenCtxStreamCreate", &pGreenStream) || !load("cuGreenCtxDestroy", &pGreenDestroy)) {
        tutti_set_cuda_error_("green-context driver entry points are not available");
        return TUTTI_ECUDA;
    }
    if (cudaSetDevice(tutti_ctx_device_(ctx)) != cudaSuccess || cudaFree(0) != cudaSuccess) {
        tutti_set_cuda_error_("cudaSetDevice failed");
        return TUTTI_ECUDA;
    }
    CUdevice dev;
    CUresult r = pDeviceGet(&dev, tutti_ctx_device_(ctx));
    if (r != CUDA_SUCCESS) return fail("cuDeviceGet", r);
    CUdevResource all, io_res, rest;
    r = pGetDevResource(dev, &all, CU_DEV_RESOURCE_TYPE_SM);
    if (r != CUDA_SUCCESS) return fail("cuDeviceGetDevResource", r);
    if (io_sms >= all.sm.smCount) return TUTTI_EINVAL;
    unsigned int n_groups = 1;
    r = pSplit(&io_res, &n_groups, &all, &rest, 0, io_sms);
    if (r != CUDA_SUCCESS || n_groups != 1) return fail("cuDevSmResourceSplitByCount", r);
    PartitionState *ps = new PartitionState();
    CUdevResourceDesc d_io, d_rest;
    r = pGenDesc(&d_io, &io_res, 1);
    if (r == CUDA_SUCCESS) r = pGenDesc(&d_rest, &rest, 1);
    if (r == CUDA_SUCCESS) r = pGreenCreate(&ps->io, d_io, dev, CU_GREEN_CTX_DEFAULT_STREAM);
    if (r == CUDA_SUCCESS) r = pGreenCreate(&ps->compute, d_rest, dev, CU_GREEN_CTX_DEFAULT_STREAM);
    if (r == CUDA_SUCCESS) r = pGreenStream(&ps->io_stream, ps->io, CU_STREAM_NON_BLOCKING, 0);
    if (r == CUDA_SUCCESS) r = pGreenStream(&ps->compute_stream, ps->compute, CU_STREAM_NON_BLOCKING, 0);
    if (r != CUDA_SUCCESS) {
        if (ps->io_stream) cudaStreamDestroy((cudaStream_t)ps->io_stream);
        if (ps->compute_stream) cudaStreamDestroy((cudaStream_t)ps->compute_stream);
        if (ps->io) pGreenDestroy(ps->io);
        if (ps->compute) pGreenDestroy(ps->compute);
        delete ps;
        return fail("green context setup", r);
    }
    *slot = ps;
    *io_stream = ps->io_stream;
    *compute_stream = ps->compute_stream;
    if (io_sms_got) *io_sms_got = io_res.sm.smCount;
    if (compute_sms_got) *compute_sms_got = rest.sm.smCount;
    return TUTTI_OK;
}

extern "C" int tutti_sm_partition_destroy(tutti_ctx_t *ctx) {
    if (!ctx) return TUTTI_EINVAL;
    void **slot = tutti_ctx_partition_slot_(ctx);
    if (!*slot) return TUTTI_OK;
    PartitionState *ps = static_cast<PartitionState *>(*slot);
    CUresult (*pGreenDestroy)(CUgreenCtx) = nullptr;
    cudaStreamSynchronize((cudaStream_t)ps->io_stream);
    cudaStreamSynchronize((cudaStream_t)ps->compute_stream);
    cudaStreamDestroy((cudaStream_t)ps->io_stream);
    cudaStreamDestroy((cudaStream_t)ps->compute_stream);
    if (load("cuGreenCtxDestroy", &pGreenDestroy)) {
        pGreenDestroy(ps->io);
        pGreenDestroy(ps->compute);
    }
    delete ps;
    *slot = nullptr;
    return TUTTI_OK;
}
