// The two storage formats that HAC and sHAC are measured against, with their products on the device:
// the index map (Sect. III-C.1: a vector of the k distinct values and one small pointer per weight) and
// plain CSC (Sect. IV-A: nz, ri, cb).  Neither is entropy coded, so a weight costs one table lookup (index
// map) or one gather of x (CSC) and both kernels are plain streaming reductions: one warp per column,
// 128-bit loads of the pointers, the sum finished with a fixed shuffle tree.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>

#include "hac_internal.h"

namespace hacb200 {

namespace {

constexpr int kCmpThreads = 256;
constexpr int kCmpWarps = kCmpThreads / 32;
constexpr int kCmpBatchTile = 4;                 // inputs that share one pass over a column
constexpr int kCodebookCopies = 32;              // one copy of the 256-entry codebook per shared-memory bank

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct Strides {
    int64_t x_i, x_b, y_j, y_b;
};

// Index map with one byte per weight.  The codebook sits in shared memory once per bank (entry e of lane l at
// [e * 32 + l]), so the 32 lookups of a warp never collide whatever the pointers are.
template <int kB>
__global__ void __launch_bounds__(kCmpThreads)
index_map8_kernel(const uint8_t* __restrict__ index, const float* __restrict__ codebook, int k, int64_t n, int64_t m,
                  const float* __restrict__ x, int batch, Strides st, float* __restrict__ y) {
    extern __shared__ float cb_s[];
    for (int e = threadIdx.x; e < 256 * kCodebookCopies; e += kCmpThreads) {
        const int entry = e / kCodebookCopies;
        cb_s[e] = entry < k ? codebook[entry] : 0.0f;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const float* mine = cb_s + lane;
    const int64_t warp = (int64_t)blockIdx.x * kCmpWarps + (threadIdx.x >> 5);
    const int64_t warps = (int64_t)gridDim.x * kCmpWarps;
    const bool wide = (n % 16) == 0 && (reinterpret_cast<uintptr_t>(index) % 16) == 0;
    for (int64_t j = warp; j < m; j += warps) {
        const uint8_t* col = index + j * n;
        for (int b0 = 0; b0 < batch; b0 += kB) {
            float acc[kB];
#pragma unroll
            for (int b = 0; b < kB; ++b) acc[b] = 0.0f;
            if (wide) {
                for (int64_t i = (int64_t)lane * 16; i < n; i += 32 * 16) {
                    const uint4 q = __ldg(reinterpret_cast<const uint4*>(col + i));
                    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const float w = mine[((w4[t >> 2] >> (8 * (t & 3))) & 0xffu) * kCodebookCopies];
#pragma unroll
                        for (int b = 0; b < kB; ++b)
                            if (b0 + b < batch) acc[b] = fmaf(w, __ldg(x + (i + t) * st.x_i + (int64_t)(b0 + b) * st.x_b), acc[b]);
                    }
                }
            } else {
                for (int64_t i = lane; i < n; i += 32) {
                    const float w = mine[(uint32_t)col[i] * kCodebookCopies];
#pragma unroll
                    for (int b = 0; b < kB; ++b)
                        if (b0 + b < batch) acc[b] = fmaf(w, __ldg(x + i * st.x_i + (int64_t)(b0 + b) * st.x_b), acc[b]);
                }
            }
#pragma unroll
            for (int b = 0; b < kB; ++b) {
                const float s = warp_sum(acc[b]);
                if (lane == 0 && b0 + b < batch) y[j * st.y_j + (int64_t)(b0 + b) * st.y_b] = s;
            }
        }
    }
}

// One input, x contiguous and small enough for shared memory: x is staged once per block, a lane takes sixteen consecutive
// pointers (one 128-bit load, two of them in flight) and the sixteen matching elements of x.  x is stored with four padding
// words after every sixteen, so that the 128-bit reads of the eight lanes of a quarter-warp, 16 elements apart, fall on
// disjoint banks.
constexpr int kVecThreads = 512;
constexpr int kVecWarps = kVecThreads / 32;
__host__ __device__ constexpr int64_t padded_x(int64_t i) { return i + (i >> 4) * 4; }

__global__ void __launch_bounds__(kVecThreads)
index_map8_vec_kernel(const uint8_t* __restrict__ index, const float* __restrict__ codebook, int k, int64_t n, int64_t m,
                      const float* __restrict__ x, float* __restrict__ y, int64_t y_stride_j) {
    extern __shared__ __align__(16) float smem[];
    float* cb_s = smem;                                   // [256][32]
    float* x_s = smem + 256 * kCodebookCopies;            // [padded_x(n)]
    for (int e = threadIdx.x; e < 256 * kCodebookCopies; e += kVecThreads) {
        const int entry = e / kCodebookCopies;
        cb_s[e] = entry < k ? codebook[entry] : 0.0f;
    }
    for (int64_t i = threadIdx.x; i < n; i += kVecThreads) x_s[padded_x(i)] = __ldg(x + i);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const float* mine = cb_s + lane;
    const int64_t warp = (int64_t)blockIdx.x * kVecWarps + (threadIdx.x >> 5);
    const int64_t warps = (int64_t)gridDim.x * kVecWarps;
    const int64_t groups = n / 16;                        // n is a multiple of 16 here
    for (int64_t j = warp; j < m; j += warps) {
        const uint4* col = reinterpret_cast<const uint4*>(index + j * n);
        float acc0 = 0.0f, acc1 = 0.0f;
        for (int64_t g0 = lane; g0 < groups; g0 += 2 * 32) {
            uint4 p[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) p[u] = g0 + 32 * u < groups ? __ldg(col + g0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (g0 + 32 * u < groups) {
                    const float* xg = x_s + 20 * (g0 + 32 * u);
                    const uint32_t w4[4] = {p[u].x, p[u].y, p[u].z, p[u].w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float4 xv = *reinterpret_cast<const float4*>(xg + 4 * t);
                        acc0 = fmaf(mine[(w4[t] & 0xffu) * kCodebookCopies], xv.x, acc0);
                        acc1 = fmaf(mine[((w4[t] >> 8) & 0xffu) * kCodebookCopies], xv.y, acc1);
                        acc0 = fmaf(mine[((w4[t] >> 16) & 0xffu) * kCodebookCopies], xv.z, acc0);
                        acc1 = fmaf(mine[(w4[t] >> 24) * kCodebookCopies], xv.w, acc1);
                    }
                }
            }
        }
        const float s = warp_sum(acc0 + acc1);
        if (lane == 0) y[j * y_stride_j] = s;
    }
}

// CSC, one input, x staged in shared memory and gathered from there.
__global__ void __launch_bounds__(kVecThreads)
csc_vec_kernel(const float* __restrict__ nz, const uint32_t* __restrict__ ri, const uint32_t* __restrict__ cb, int64_t n,
               int64_t m, const float* __restrict__ x, float* __restrict__ y, int64_t y_stride_j) {
    extern __shared__ __align__(16) float smem[];
    for (int64_t i = threadIdx.x; i < n; i += kVecThreads) smem[i] = __ldg(x + i);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * kVecWarps + (threadIdx.x >> 5);
    const int64_t warps = (int64_t)gridDim.x * kVecWarps;
    for (int64_t j = warp; j < m; j += warps) {
        const uint32_t lo = __ldg(cb + j), hi = __ldg(cb + j + 1);
        float acc0 = 0.0f, acc1 = 0.0f;
        for (uint32_t p0 = lo + lane; p0 < hi; p0 += 4 * 32) {
            float w[4];
            uint32_t r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool in = p0 + 32 * u < hi;
                w[u] = in ? __ldg(nz + p0 + 32 * u) : 0.0f;
                r[u] = in ? __ldg(ri + p0 + 32 * u) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; u += 2) {
                acc0 = fmaf(w[u], r[u] < n ? smem[r[u]] : 0.0f, acc0);
                acc1 = fmaf(w[u + 1], r[u + 1] < n ? smem[r[u + 1]] : 0.0f, acc1);
            }
        }
        const float s = warp_sum(acc0 + acc1);
        if (lane == 0) y[j * y_stride_j] = s;
    }
}

// Index map with two bytes per weight (more than 256 values): the codebook stays in global memory and is
// read through the read-only cache.  A pointer at or beyond k reads the last entry.
template <int kB>
__global__ void __launch_bounds__(kCmpThreads)
index_map16_kernel(const uint16_t* __restrict__ index, const float* __restrict__ codebook, int k, int64_t n, int64_t m,
                   const float* __restrict__ x, int batch, Strides st, float* __restrict__ y) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * kCmpWarps + (threadIdx.x >> 5);
    const int64_t warps = (int64_t)gridDim.x * kCmpWarps;
    const bool wide = (n % 8) == 0 && (reinterpret_cast<uintptr_t>(index) % 16) == 0;
    const uint32_t last = (uint32_t)(k - 1);
    for (int64_t j = warp; j < m; j += warps) {
        const uint16_t* col = index + j * n;
        for (int b0 = 0; b0 < batch; b0 += kB) {
            float acc[kB];
#pragma unroll
            for (int b = 0; b < kB; ++b) acc[b] = 0.0f;
            if (wide) {
                for (int64_t i = (int64_t)lane * 8; i < n; i += 32 * 8) {
                    const uint4 q = __ldg(reinterpret_cast<const uint4*>(col + i));
                    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const uint32_t p = (w4[t >> 1] >> (16 * (t & 1))) & 0xffffu;
                        const float w = __ldg(codebook + min(p, last));
#pragma unroll
                        for (int b = 0; b < kB; ++b)
                            if (b0 + b < batch) acc[b] = fmaf(w, __ldg(x + (i + t) * st.x_i + (int64_t)(b0 + b) * st.x_b), acc[b]);
                    }
                }
            } else {
                for (int64_t i = lane; i < n; i += 32) {
                    const float w = __ldg(codebook + min((uint32_t)col[i], last));
#pragma unroll
                    for (int b = 0; b < kB; ++b)
                        if (b0 + b < batch) acc[b] = fmaf(w, __ldg(x + i * st.x_i + (int64_t)(b0 + b) * st.x_b), acc[b]);
                }
            }
#pragma unroll
            for (int b = 0; b < kB; ++b) {
                const float s = warp_sum(acc[b]);
                if (lane == 0 && b0 + b < batch) y[j * st.y_j + (int64_t)(b0 + b) * st.y_b] = s;
            }
        }
    }
}

// CSC: the stored entries of column j are nz[cb[j] .. cb[j+1]) with rows ri[...]; lanes take them in turn.
// A row at or beyond n (a corrupt ri) contributes nothing.
template <int kB>
__global__ void __launch_bounds__(kCmpThreads)
csc_kernel(const float* __restrict__ nz, const uint32_t* __restrict__ ri, const uint32_t* __restrict__ cb, int64_t n,
           int64_t m, const float* __restrict__ x, int batch, Strides st, float* __restrict__ y) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * kCmpWarps + (threadIdx.x >> 5);
    const int64_t warps = (int64_t)gridDim.x * kCmpWarps;
    for (int64_t j = warp; j < m; j += warps) {
        const uint32_t lo = __ldg(cb + j), hi = __ldg(cb + j + 1);
        for (int b0 = 0; b0 < batch; b0 += kB) {
            float acc[kB];
#pragma unroll
            for (int b = 0; b < kB; ++b) acc[b] = 0.0f;
            for (uint32_t p = lo + lane; p < hi; p += 32) {
                const float w = __ldg(nz + p);
                const uint32_t i = __ldg(ri + p);
                if (i < n) {
#pragma unroll
                    for (int b = 0; b < kB; ++b)
                        if (b0 + b < batch) acc[b] = fmaf(w, __ldg(x + (int64_t)i * st.x_i + (int64_t)(b0 + b) * st.x_b), acc[b]);
                }
            }
#pragma unroll
            for (int b = 0; b < kB; ++b) {
                const float s = warp_sum(acc[b]);
                if (lane == 0 && b0 + b < batch) y[j * st.y_j + (int64_t)(b0 + b) * st.y_b] = s;
            }
        }
    }
}

int cuda_error(cudaError_t e, const char* what) {
    set_last_cuda_error(std::string(what) + ": " + cudaGetErrorString(e));
    return HAC_ERR_CUDA;
}

// Enough blocks to fill the device a few times over, never more than there are columns to hand out.
int device_limits(int* sms, int* smem_optin) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    return e == cudaSuccess ? HAC_OK : cuda_error(e, "cudaDeviceGetAttribute");
}

int grid_for(int64_t m, int* out) {
    int sms = 0, smem = 0;
    if (int rc = device_limits(&sms, &smem)) return rc;
    const int64_t want = (m + kCmpWarps - 1) / kCmpWarps;
    *out = (int)std::max<int64_t>(1, std::min<int64_t>(want, (int64_t)sms * 8));
    return HAC_OK;
}

// Launch shape of the kernels that stage x: as many blocks per SM as the shared memory allows (at most 4), the columns dealt
// to their warps.  Returns false when x does not fit.
bool staged_x_shape(int64_t m, size_t smem_bytes, int sms, int smem_optin, int* grid) {
    if (smem_bytes > (size_t)smem_optin) return false;
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(4, ((size_t)228 * 1024) / (smem_bytes + 1024)));
    const int64_t want = (m + kVecWarps - 1) / kVecWarps;
    *grid = (int)std::max<int64_t>(1, std::min<int64_t>(want, (int64_t)sms * per_sm));
    return true;
}

bool finite_and_normal_zero(float& v) {
    if (!std::isfinite(v)) return false;
    if (v == 0.0f) v = 0.0f;                          // -0.0 counts as 0
    return true;
}

}  // namespace

}  // namespace hacb200

using namespace hacb200;

extern "C" {

int hac_index_map_encode(const float* Wq, int64_t n, int64_t m, int64_t ldw, int index_bits, void* index_colmajor,
                         float* codebook, int* k_out) {
    if (!Wq || !index_colmajor || !codebook || !k_out || n < 1 || m < 1 || ldw < m || (index_bits != 8 && index_bits != 16))
        return HAC_ERR_INVALID_ARG;
    const size_t cap = (size_t)1 << index_bits;
    std::vector<float> values;
    try {
        values.reserve((size_t)n * (size_t)m);
        for (int64_t i = 0; i < n; ++i)
            for (int64_t j = 0; j < m; ++j) {
                float v = Wq[i * ldw + j];
                if (!finite_and_normal_zero(v)) return HAC_ERR_NONFINITE_INPUT;
                values.push_back(v);
            }
        std::vector<float> c(values);
        std::sort(c.begin(), c.end());
        c.erase(std::unique(c.begin(), c.end()), c.end());
        if (c.size() > cap) return HAC_ERR_K_TOO_LARGE;
        for (size_t e = 0; e < c.size(); ++e) codebook[e] = c[e];
        *k_out = (int)c.size();
        for (int64_t i = 0; i < n; ++i)
            for (int64_t j = 0; j < m; ++j) {
                const size_t p = (size_t)(std::lower_bound(c.begin(), c.end(), values[(size_t)(i * m + j)]) - c.begin());
                if (index_bits == 8) static_cast<uint8_t*>(index_colmajor)[j * n + i] = (uint8_t)p;
                else static_cast<uint16_t*>(index_colmajor)[j * n + i] = (uint16_t)p;
            }
    } catch (const std::bad_alloc&) {
        return HAC_ERR_ALLOC;
    }
    return HAC_OK;
}

int hac_index_map_dot(const void* index_dev, int index_bits, const float* codebook_dev, int k, int64_t n, int64_t m,
                      const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
                      int64_t y_stride_j, int64_t y_stride_b, void* cuda_stream) {
    if (!index_dev || !codebook_dev || !x || !y || n < 1 || m < 1 || batch < 1 || batch > INT32_MAX || k < 1 ||
        (index_bits != 8 && index_bits != 16) || k > (1 << index_bits))
        return HAC_ERR_INVALID_ARG;
    int grid = 0;
    if (int rc = grid_for(m, &grid)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const Strides st{x_stride_i, x_stride_b, y_stride_j, y_stride_b};
    if (index_bits == 8 && batch == 1 && x_stride_i == 1 && n % 16 == 0 && reinterpret_cast<uintptr_t>(index_dev) % 16 == 0) {
        int sms = 0, optin = 0, vgrid = 0;
        if (int rc = device_limits(&sms, &optin)) return rc;
        const size_t smem = ((size_t)256 * kCodebookCopies + (size_t)padded_x(n)) * sizeof(float);
        if (staged_x_shape(m, smem, sms, optin, &vgrid)) {
            cudaError_t e = cudaFuncSetAttribute(index_map8_vec_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return cuda_error(e, "cudaFuncSetAttribute");
            index_map8_vec_kernel<<<vgrid, kVecThreads, smem, s>>>(static_cast<const uint8_t*>(index_dev), codebook_dev, k, n, m, x,
                                                                    y, y_stride_j);
            e = cudaGetLastError();
            return e == cudaSuccess ? HAC_OK : cuda_error(e, "index map kernel launch");
        }
    }
    if (index_bits == 8) {
        const size_t smem = (size_t)256 * kCodebookCopies * sizeof(float);
        auto launch = [&](auto kern) -> int {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return cuda_error(e, "cudaFuncSetAttribute");
            kern<<<grid, kCmpThreads, smem, s>>>(static_cast<const uint8_t*>(index_dev), codebook_dev, k, n, m, x, (int)batch,
                                                 st, y);
            return HAC_OK;
        };
        if (int rc = batch == 1 ? launch(index_map8_kernel<1>) : launch(index_map8_kernel<kCmpBatchTile>)) return rc;
    } else {
        if (batch == 1)
            index_map16_kernel<1><<<grid, kCmpThreads, 0, s>>>(static_cast<const uint16_t*>(index_dev), codebook_dev, k, n, m,
                                                               x, (int)batch, st, y);
        else
            index_map16_kernel<kCmpBatchTile><<<grid, kCmpThreads, 0, s>>>(static_cast<const uint16_t*>(index_dev),
                                                                           codebook_dev, k, n, m, x, (int)batch, st, y);
    }
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? HAC_OK : cuda_error(e, "index map kernel launch");
}

int shac_csc_encode(const float* Wq, int64_t n, int64_t m, int64_t ldw, float* nz, uint32_t* ri, uint32_t* cb,
                    int64_t capacity, int64_t* q_out) {
    if (!Wq || !q_out || n < 1 || m < 1 || ldw < m || n > (int64_t)UINT32_MAX) return HAC_ERR_INVALID_ARG;
    int64_t q = 0;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t j = 0; j < m; ++j) {
            float v = Wq[i * ldw + j];
            if (!finite_and_normal_zero(v)) return HAC_ERR_NONFINITE_INPUT;
            q += v != 0.0f;
        }
    *q_out = q;
    if (q > (int64_t)UINT32_MAX) return HAC_ERR_OFFSET_OVERFLOW;
    if (!nz && !ri && !cb) return HAC_OK;                       // size query
    if (!nz || !ri || !cb) return HAC_ERR_INVALID_ARG;
    if (capacity < q) return HAC_ERR_BUFFER_TOO_SMALL;
    int64_t p = 0;
    for (int64_t j = 0; j < m; ++j) {
        cb[j] = (uint32_t)p;
        for (int64_t i = 0; i < n; ++i) {
            const float v = Wq[i * ldw + j];
            if (v != 0.0f) { nz[p] = v; ri[p] = (uint32_t)i; ++p; }
        }
    }
    cb[m] = (uint32_t)p;
    return HAC_OK;
}

int shac_csc_dot(const float* nz_dev, const uint32_t* ri_dev, const uint32_t* cb_dev, int64_t n, int64_t m, const float* x,
                 int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y, int64_t y_stride_j, int64_t y_stride_b,
                 void* cuda_stream) {
    if (!cb_dev || !x || !y || n < 1 || m < 1 || batch < 1 || batch > INT32_MAX) return HAC_ERR_INVALID_ARG;
    int grid = 0;
    if (int rc = grid_for(m, &grid)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const Strides st{x_stride_i, x_stride_b, y_stride_j, y_stride_b};
    if (batch == 1 && x_stride_i == 1) {
        int sms = 0, optin = 0, vgrid = 0;
        if (int rc = device_limits(&sms, &optin)) return rc;
        const size_t smem = (size_t)n * sizeof(float);
        if (staged_x_shape(m, smem, sms, optin, &vgrid)) {
            cudaError_t e = cudaFuncSetAttribute(csc_vec_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return cuda_error(e, "cudaFuncSetAttribute");
            csc_vec_kernel<<<vgrid, kVecThreads, smem, s>>>(nz_dev, ri_dev, cb_dev, n, m, x, y, y_stride_j);
            e = cudaGetLastError();
            return e == cudaSuccess ? HAC_OK : cuda_error(e, "CSC kernel launch");
        }
    }
    if (batch == 1) csc_kernel<1><<<grid, kCmpThreads, 0, s>>>(nz_dev, ri_dev, cb_dev, n, m, x, (int)batch, st, y);
    else csc_kernel<kCmpBatchTile><<<grid, kCmpThreads, 0, s>>>(nz_dev, ri_dev, cb_dev, n, m, x, (int)batch, st, y);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? HAC_OK : cuda_error(e, "CSC kernel launch");
}

}  // extern "C"
