// Stand-alone timing loop over the encoder's per-group vector passes (no memory traffic in the loop):
// pass A (threshold split + min / max), pass B for the first lower candidate with the FMA quotient at
// two levels, byte assembly + 8 x 32 bit transpose.  Run under `ncu --metrics smsp__inst_executed.sum,
// sm__inst_executed_pipe_alu.sum,sm__inst_executed_pipe_fma.sum,gpu__time_duration.sum` it gives the
// instructions per element and the pipe mix of each pass: the ceiling that the full kernel's
// arithmetic sets, apart from everything the kernel does around the passes.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -fmad=false -ftz=false -prec-div=true \
//        -I include -I paper_2511_04002_b200/csrc paper_2511_04002_b200/csrc/microbench/passes.cu -o passes
//
// Every kernel processes 148 * 4 * 256 threads x 64 iterations x 32 elements; k_empty is the loop's own
// cost (the pseudo-random refresh of the inputs) and is to be subtracted.
#include <cstdio>
#include <vector>

#include "../tsq_encode.cu"

namespace tsq {
namespace {
constexpr int kIters = 64;

__device__ __forceinline__ void load16(const uint4* in, uint32_t (&x)[16]) {
  const uint4* q = in + (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  for (int j = 0; j < 4; ++j) {
    const uint4 c = q[j];
    x[4 * j] = c.x, x[4 * j + 1] = c.y, x[4 * j + 2] = c.z, x[4 * j + 3] = c.w;
  }
}
__device__ __forceinline__ uint32_t refresh(uint32_t (&x)[16]) {
  uint32_t acc = 0;
  for (int i = 0; i < 16; ++i) {
    x[i] = (x[i] * 1664525u + 1013904223u) & 0xbfffbfffu;  // finite bf16 pairs
    acc ^= x[i];
  }
  return acc;
}

__global__ void k_empty(const uint4* in, uint32_t* out) {
  uint32_t x[16], acc = 0;
  load16(in, x);
  for (int it = 0; it < kIters; ++it) acc ^= refresh(x);
  out[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}
__global__ void k_pass_a(const uint4* in, uint32_t* out, uint32_t thr2) {
  uint32_t x[16], acc = 0, mn = 0x7f807f80u, mx = 0;
  load16(in, x);
  for (int it = 0; it < kIters; ++it) {
    acc ^= refresh(x);
    acc += split_group<true>(x, 4, thr2, mn, mx);
  }
  out[blockIdx.x * blockDim.x + threadIdx.x] = acc + mn + mx;
}
__global__ void k_pass_b(const uint4* in, uint32_t* out, float mmax) {
  uint32_t x[16], acc = 0;
  load16(in, x);
  const Level top = make_level(0.f, mmax, 8), low = make_level(0.f, mmax, 4);
  for (int it = 0; it < kIters; ++it) {
    acc ^= refresh(x);
    uint32_t tb[8], ql[8];
    acc += distortion_first<true, false>(x, top, low, 4, tb, ql);
    for (int i = 0; i < 8; ++i) acc ^= tb[i];
  }
  out[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}
__global__ void k_pass_b_c(const uint4* in, uint32_t* out, float mmax) {
  uint32_t x[16], acc = 0;
  load16(in, x);
  const Level top = make_level(0.f, mmax, 8), low = make_level(0.f, mmax, 4);
  for (int it = 0; it < kIters; ++it) {
    acc ^= refresh(x);
    uint32_t tb[8], ql[8], r[8];
    acc += distortion_first<true, false>(x, top, low, 4, tb, ql);
    planes_of_bytes(tb, r);
    for (int i = 0; i < 8; ++i) acc ^= r[i];
  }
  out[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}
}  // namespace
}  // namespace tsq

using namespace tsq;

int main() {
  const int blocks = 148 * 4, threads = 256, n = blocks * threads;
  uint4* in;
  uint32_t* out;
  if (cudaMalloc(&in, sizeof(uint4) * 4 * n) != cudaSuccess || cudaMalloc(&out, 4 * n) != cudaSuccess) return 1;
  std::vector<uint32_t> h(16 * n);
  uint32_t s = 12345;
  for (auto& v : h) {
    s = s * 1664525u + 1013904223u;
    v = s & 0x3fff3fffu;
  }
  cudaMemcpy(in, h.data(), h.size() * 4, cudaMemcpyHostToDevice);
  const float mmax = 7.5f;
  const uint32_t thr2 = 0x41004100u;  // bf16 8.0 in both halves
  for (int rep = 0; rep < 2; ++rep) {
    k_empty<<<blocks, threads>>>(in, out);
    k_pass_a<<<blocks, threads>>>(in, out, thr2);
    k_pass_b<<<blocks, threads>>>(in, out, mmax);
    k_pass_b_c<<<blocks, threads>>>(in, out, mmax);
  }
  const cudaError_t e = cudaDeviceSynchronize();
  std::printf("%s: %d threads x %d iterations x 32 elements per kernel\n", cudaGetErrorString(e), n, kIters);
  return e != cudaSuccess;
}
