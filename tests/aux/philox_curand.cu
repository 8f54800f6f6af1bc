// Third implementation of Philox4x32-10 for the tests: the device function of cuRAND's header,
// called for n (counter, key) pairs.  Built by the test with nvcc; not part of the library.
#include <cuda_runtime.h>
#include <curand_kernel.h>
#include <stdint.h>

__global__ void k_curand_philox(const uint32_t *ctr, uint32_t k0, uint32_t k1, uint32_t *out, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint4 c = make_uint4(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3]);
    const uint4 r = curand_Philox4x32_10(c, make_uint2(k0, k1));
    out[4 * i] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
}

extern "C" int curand_philox_host(const uint32_t *ctr, uint32_t k0, uint32_t k1, uint32_t *out, int n)
{
    uint32_t *d_ctr = nullptr, *d_out = nullptr;
    if (cudaMalloc(&d_ctr, sizeof(uint32_t) * 4 * n) != cudaSuccess) return 1;
    if (cudaMalloc(&d_out, sizeof(uint32_t) * 4 * n) != cudaSuccess) { cudaFree(d_ctr); return 1; }
    cudaMemcpy(d_ctr, ctr, sizeof(uint32_t) * 4 * n, cudaMemcpyHostToDevice);
    k_curand_philox<<<(n + 127) / 128, 128>>>(d_ctr, k0, k1, d_out, n);
    const cudaError_t e = cudaMemcpy(out, d_out, sizeof(uint32_t) * 4 * n, cudaMemcpyDeviceToHost);
    cudaFree(d_ctr); cudaFree(d_out);
    return e == cudaSuccess ? 0 : 2;
}
