// rago_index_load_pq4: an index whose product quantiser uses 4-bit codes (16 codewords per sub-space, two codes
// per byte).  Two adjacent sub-spaces with their 16 x 16 code combinations are one 8-bit sub-space whose 256
// codewords are the concatenations, and the packed byte is its code.  So the loader writes that paired codebook
// once and hands it to the ordinary loader: table build, scan and selection are the 8-bit kernels, one table
// look-up now covers two sub-quantisers, and every byte read from the lists carries two of them.
#include "common.cuh"

namespace rago {

// pair[j][byte][0 .. ds) = cb4[2j][byte & 15], pair[j][byte][ds .. 2 ds) = cb4[2j + 1][byte >> 4]
__global__ void pair_codebooks_kernel(const float* __restrict__ cb4, int M, int ds, float* __restrict__ pair) {
    const size_t total = (size_t)M * 256 * 2 * ds;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(e % (2 * ds));
        const int byte = (int)((e / (2 * ds)) % 256);
        const int j = (int)(e / ((size_t)2 * ds * 256));
        const int sub = 2 * j + (t >= ds);
        const int code = t >= ds ? byte >> 4 : byte & 15;
        pair[e] = cb4[((size_t)sub * 16 + code) * ds + (t >= ds ? t - ds : t)];
    }
}

}  // namespace rago

using namespace rago;

extern "C" rago_status rago_index_load_pq4(rago_index** out, const void* coarse_centroids, rago_dtype coarse_dtype,
                                           const float* pq4_codebooks, const uint8_t* packed_codes,
                                           const int64_t* list_offsets, const int64_t* ids, int64_t N, int32_t d,
                                           int32_t nlist, int32_t M4, rago_metric metric, void* cuda_stream) {
    if (!out) { set_error("out is null"); return RAGO_EINVAL; }
    *out = nullptr;
    if (!pq4_codebooks) { set_error("null index array"); return RAGO_EINVAL; }
    if (M4 <= 0 || d <= 0 || M4 % 2 != 0 || d % M4 != 0) {
        set_error("M4 = %d must be positive and even, and d = %d a multiple of it", M4, d);
        return RAGO_EINVAL;
    }
    if (reinterpret_cast<uintptr_t>(pq4_codebooks) % 16) { set_error("pq4_codebooks needs 16-byte alignment"); return RAGO_EALIGN; }
    const int M = M4 / 2, ds = d / M4;
    float* pair = nullptr;
    cudaError_t e = cudaMalloc(&pair, (size_t)M * 256 * 2 * ds * sizeof(float));
    if (e != cudaSuccess) { cudaGetLastError(); set_error("device allocation of the paired codebook failed"); return RAGO_ENOMEM; }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t total = (size_t)M * 256 * 2 * ds;
    pair_codebooks_kernel<<<(unsigned)((total + 255) / 256 < 1024 ? (total + 255) / 256 : 1024), 256, 0, s>>>(
        pq4_codebooks, M, ds, pair);
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) { cudaFree(pair); set_error("pair_codebooks_kernel: %s", cudaGetErrorString(e)); return RAGO_ECUDA; }
    // The ordinary loader derives everything it keeps (transposed codebook, per-vector terms) from the
    // codebook before it returns, and it returns with the stream drained: the paired copy can go then.
    const rago_status st = rago_index_load(out, coarse_centroids, coarse_dtype, pair, packed_codes, list_offsets, ids,
                                           N, d, nlist, M, metric, cuda_stream);
    cudaStreamSynchronize(s);
    cudaFree(pair);
    if (st == RAGO_OK) reinterpret_cast<IndexImpl*>(*out)->codebooks = nullptr;
    return st;
}
