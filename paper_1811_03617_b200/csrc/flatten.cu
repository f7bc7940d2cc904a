// The flatten order of a convolutional layer's gradient (Section 2, figure on flattening and slicing): the F
// gradients of one position (h, w, depth) next to each other, positions visited depth first, then width, then
// height -- against the framework's [F][D][H][W].  With x = h * W + w, X = H * W and C = D * X:
//     flat[(x * D + dep) * F + f] = framework[f * C + dep * X + x]
// i.e. the transpose of an F x C matrix whose columns are then taken in the order (x, dep) instead of (dep, x).
// Tiles of 64 filters x 64 columns go through shared memory, so that both sides move 256-byte rows and a thread
// has sixteen loads in flight.
#include "gvq_internal.h"

namespace gvq {
namespace {

// grid (ceil(C / 64), ceil(F / 64)), block (64, 4).  INVERSE: flat -> framework.
template <bool INVERSE>
__global__ void __launch_bounds__(256) flatten_kernel(int F, int D, int X, const float *__restrict__ src, float *__restrict__ dst)
{
    __shared__ float tile[64][65];
    const int C = D * X;
    const int c0 = blockIdx.x * 64, f0 = blockIdx.y * 64;
    const int tx = threadIdx.x, ty = threadIdx.y;
    // column c = dep * X + x of the framework layout sits at row x * D + dep of the flat one
    auto flat_row = [&](int c) { const int dep = c / X, x = c - dep * X; return x * D + dep; };
    if (!INVERSE) {
        for (int i = ty; i < 64; i += 4) {   // read framework rows (f), columns c contiguous
            const int f = f0 + i, c = c0 + tx;
            if (f < F && c < C) tile[i][tx] = src[(size_t)f * C + c];
        }
        __syncthreads();
        for (int i = ty; i < 64; i += 4) {   // write flat rows (one per column c), filters contiguous
            const int c = c0 + i, f = f0 + tx;
            if (c < C && f < F) dst[(size_t)flat_row(c) * F + f] = tile[tx][i];
        }
    } else {
        for (int i = ty; i < 64; i += 4) {
            const int c = c0 + i, f = f0 + tx;
            if (c < C && f < F) tile[tx][i] = src[(size_t)flat_row(c) * F + f];
        }
        __syncthreads();
        for (int i = ty; i < 64; i += 4) {
            const int f = f0 + i, c = c0 + tx;
            if (f < F && c < C) dst[(size_t)f * C + c] = tile[i][tx];
        }
    }
}

}  // namespace

cudaError_t launch_flatten(cudaStream_t st, int F, int D, int X, const float *src, float *dst, bool inverse)
{
    const long long C = (long long)D * X;
    const dim3 grid((unsigned)((C + 63) / 64), (unsigned)((F + 63) / 64)), block(64, 4);
    if (inverse) flatten_kernel<true><<<grid, block, 0, st>>>(F, D, X, src, dst);
    else flatten_kernel<false><<<grid, block, 0, st>>>(F, D, X, src, dst);
    return cudaGetLastError();
}

}  // namespace gvq
