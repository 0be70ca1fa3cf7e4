// Device-side dispatch through a CUDA-graph conditional SWITCH node (paper Section IV-C) and
// the data-dependent dispatch microbenchmark of the paper's Table III.
#include <vector>

#include "common.cuh"

namespace {

__global__ void mb_producer_kernel(int* value, int seed, cudaGraphConditionalHandle handle, int use_handle) {
  const int v = (seed * 1103515245 + 12345) & 1;  // a value only the GPU computes
  *value = v;
  if (use_handle) cudaGraphSetConditional(handle, static_cast<unsigned int>(v));
}
__global__ void mb_follow_a_kernel(int* out) { out[0] += 1; }
__global__ void mb_follow_b_kernel(int* out) { out[1] += 1; }

#define MB_CUDA(expr)                       \
  do {                                      \
    if ((expr) != cudaSuccess) goto fail;   \
  } while (0)

}  // namespace

extern "C" int damoe_dispatch_microbench(int device, int iters, float* us) {
  if (!us || iters < 1) return DAMOE_ERR_INVALID_ARG;
  int* d_val = nullptr;
  int* d_out = nullptr;
  int* h_val = nullptr;
  cudaStream_t st = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaGraph_t g_cond = nullptr, g_fixed = nullptr;
  cudaGraphExec_t x_cond = nullptr, x_fixed = nullptr;
  int rc = DAMOE_ERR_CUDA;
  float ms = 0.f;
  {
    MB_CUDA(cudaSetDevice(device));
    MB_CUDA(cudaMalloc(&d_val, sizeof(int)));
    MB_CUDA(cudaMalloc(&d_out, 2 * sizeof(int)));
    MB_CUDA(cudaMemset(d_out, 0, 2 * sizeof(int)));
    MB_CUDA(cudaMallocHost(&h_val, sizeof(int)));
    MB_CUDA(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    MB_CUDA(cudaEventCreate(&e0));
    MB_CUDA(cudaEventCreate(&e1));

    // (2) fixed graph: producer -> follow-up A
    MB_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    mb_producer_kernel<<<1, 1, 0, st>>>(d_val, 1, 0, 0);
    mb_follow_a_kernel<<<1, 1, 0, st>>>(d_out);
    MB_CUDA(cudaStreamEndCapture(st, &g_fixed));
    MB_CUDA(cudaGraphInstantiate(&x_fixed, g_fixed, 0));

    // (1) conditional graph: producer sets the handle, SWITCH node picks body 0 or 1
    MB_CUDA(cudaGraphCreate(&g_cond, 0));
    cudaGraphConditionalHandle handle;
    MB_CUDA(cudaGraphConditionalHandleCreate(&handle, g_cond, 0, cudaGraphCondAssignDefault));
    cudaGraphNode_t n_prod, n_cond, n_body;
    int seed = 1, use = 1;
    void* pargs[4] = {&d_val, &seed, &handle, &use};
    cudaKernelNodeParams kp{};
    kp.func = reinterpret_cast<void*>(mb_producer_kernel);
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(1);
    kp.kernelParams = pargs;
    MB_CUDA(cudaGraphAddKernelNode(&n_prod, g_cond, nullptr, 0, &kp));
    cudaGraphNodeParams cp{};
    cp.type = cudaGraphNodeTypeConditional;
    cp.conditional.handle = handle;
    cp.conditional.type = cudaGraphCondTypeSwitch;
    cp.conditional.size = 2;
    MB_CUDA(cudaGraphAddNode(&n_cond, g_cond, &n_prod, 1, &cp));
    void* fargs[1] = {&d_out};
    cudaKernelNodeParams fa{};
    fa.func = reinterpret_cast<void*>(mb_follow_a_kernel);
    fa.gridDim = dim3(1);
    fa.blockDim = dim3(1);
    fa.kernelParams = fargs;
    MB_CUDA(cudaGraphAddKernelNode(&n_body, cp.conditional.phGraph_out[0], nullptr, 0, &fa));
    fa.func = reinterpret_cast<void*>(mb_follow_b_kernel);
    MB_CUDA(cudaGraphAddKernelNode(&n_body, cp.conditional.phGraph_out[1], nullptr, 0, &fa));
    MB_CUDA(cudaGraphInstantiate(&x_cond, g_cond, 0));

    // warm-up of all three paths
    for (int i = 0; i < 5; ++i) {
      MB_CUDA(cudaGraphLaunch(x_fixed, st));
      MB_CUDA(cudaGraphLaunch(x_cond, st));
    }
    MB_CUDA(cudaStreamSynchronize(st));

    // (0) copy the value to the host, branch on the CPU
    MB_CUDA(cudaEventRecord(e0, st));
    for (int i = 0; i < iters; ++i) {
      mb_producer_kernel<<<1, 1, 0, st>>>(d_val, i, 0, 0);
      MB_CUDA(cudaMemcpyAsync(h_val, d_val, sizeof(int), cudaMemcpyDeviceToHost, st));
      MB_CUDA(cudaStreamSynchronize(st));
      if (*h_val) mb_follow_b_kernel<<<1, 1, 0, st>>>(d_out);
      else mb_follow_a_kernel<<<1, 1, 0, st>>>(d_out);
    }
    MB_CUDA(cudaEventRecord(e1, st));
    MB_CUDA(cudaStreamSynchronize(st));
    MB_CUDA(cudaEventElapsedTime(&ms, e0, e1));
    us[0] = ms * 1000.f / iters;

    MB_CUDA(cudaEventRecord(e0, st));
    for (int i = 0; i < iters; ++i) MB_CUDA(cudaGraphLaunch(x_cond, st));
    MB_CUDA(cudaEventRecord(e1, st));
    MB_CUDA(cudaStreamSynchronize(st));
    MB_CUDA(cudaEventElapsedTime(&ms, e0, e1));
    us[1] = ms * 1000.f / iters;

    MB_CUDA(cudaEventRecord(e0, st));
    for (int i = 0; i < iters; ++i) MB_CUDA(cudaGraphLaunch(x_fixed, st));
    MB_CUDA(cudaEventRecord(e1, st));
    MB_CUDA(cudaStreamSynchronize(st));
    MB_CUDA(cudaEventElapsedTime(&ms, e0, e1));
    us[2] = ms * 1000.f / iters;
    rc = DAMOE_OK;
  }
fail:
  if (x_cond) cudaGraphExecDestroy(x_cond);
  if (x_fixed) cudaGraphExecDestroy(x_fixed);
  if (g_cond) cudaGraphDestroy(g_cond);
  if (g_fixed) cudaGraphDestroy(g_fixed);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (st) cudaStreamDestroy(st);
  if (h_val) cudaFreeHost(h_val);
  if (d_out) cudaFree(d_out);
  if (d_val) cudaFree(d_val);
  return rc;
}
