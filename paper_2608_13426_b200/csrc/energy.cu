// Column energies of a product's output accumulated where the output is produced (the authors' "jointly optimize
// selection and reduced multiplication" of the paper's closing section): the tensor-core product's epilogue writes, per
// 32-row group, the sums of squares of the rounded outputs; this kernel adds the groups up, in group order, in fp64, so
// that the next product's selection (Sec. 3.2: TopK of the column norms) needs no pass over the activations.
#include "common.cuh"

namespace rmm {
namespace {

__global__ void __launch_bounds__(256) energy_combine_kernel(const float *__restrict__ part, int64_t groups, int64_t N, float *__restrict__ energy)
{
    pdl_wait();
    const int64_t b = blockIdx.y, c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= N) return;
    const float *p = part + b * groups * N + c;
    double acc = 0.0;
    int64_t g = 0;
    for (; g + 8 <= groups; g += 8) {  // eight independent loads at a time, added in group order
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __ldcg(p + (g + i) * N);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc += (double)v[i];
    }
    for (; g < groups; ++g) acc += (double)__ldcg(p + g * N);
    energy[b * N + c] = (float)acc;
}

}  // namespace

int launch_energy_combine(const float *col_energy, int64_t batch, int64_t groups, int64_t N, float *energy, cudaStream_t stream)
{
    prof_begin("energy_combine_kernel", stream);
    launch_kernel(energy_combine_kernel, dim3((unsigned)ceil_div(N, 256), (unsigned)batch), dim3(256), 0, stream, 1, col_energy, groups, N,
                  energy);
    return check_launch("energy_combine_kernel", stream);
}

}  // namespace rmm
