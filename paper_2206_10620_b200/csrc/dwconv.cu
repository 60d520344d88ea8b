// libpatconv: depthwise pattern-pruned 3x3 convolution (sm_100a) and its C ABI.
//
// Every channel has one 3x3 kernel that keeps the 4 weights of its pattern.  The layer moves
// two activations per 4 useful multiply-adds, so HBM binds it: the kernel's job is to read x
// once and write y once, in whole 16-byte (fp16: 8-byte) pieces of consecutive channels.
// A thread owns V consecutive channels of a strip of TX output pixels of one row; it walks the
// three input rows, keeps the strip's (TX-1)*stride + 3 input columns of the current row in
// registers and adds their products with the row's three taps.  Pruned taps carry weight 0 in
// the packed table [9][channels]: all nine taps run, because neighbouring channels need the
// skipped activations anyway and the arithmetic is far from binding.  Neighbouring strips and
// rows share input through L1/L2.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "dwconv.h"
#include "patconv_internal.h"

struct xgen_dwconv_packed {
    int c = 0, stride = 1;
    xgen_dtype dtype = XGEN_F32;
    int device = -1;
    int64_t surviving = 0;
    std::vector<float> w9;          // [9][c], pruned taps zero
    float *d_w9 = nullptr;
};

namespace dwconv {

struct DParams {
    const void *x; void *y; const float *bias; const float *w9;
    int n, h, w, ho, wo, c;
    int relu;
    int strips;                     // strips of TX output pixels per output row
    int items_per_row;              // strips * (c / V): threads one output row needs
    int rows_per_block;             // output rows a thread block covers (several when a row is short)
    int rows;                       // n * ho
};

template <int DT, int V>
__device__ __forceinline__ void load_vec(const void *x, unsigned elem, float (&v)[V]) {
    if constexpr (DT == XGEN_F32) {
        if constexpr (V == 4) {
            const float4 t = __ldg(reinterpret_cast<const float4 *>(static_cast<const float *>(x) + elem));
            v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
        } else v[0] = __ldg(static_cast<const float *>(x) + elem);
    } else {
        if constexpr (V == 4) {
            const uint2 t = __ldg(reinterpret_cast<const uint2 *>(static_cast<const __half *>(x) + elem));
            const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&t.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&t.y));
            v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
        } else v[0] = __half2float(__ldg(static_cast<const __half *>(x) + elem));
    }
}

template <int DT, int V>
__device__ __forceinline__ void store_vec(void *y, unsigned elem, const float (&v)[V]) {
    if constexpr (DT == XGEN_F32) {
        if constexpr (V == 4) *reinterpret_cast<float4 *>(static_cast<float *>(y) + elem) = make_float4(v[0], v[1], v[2], v[3]);
        else static_cast<float *>(y)[elem] = v[0];
    } else {
        if constexpr (V == 4) {
            const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
            uint2 t;
            t.x = *reinterpret_cast<const uint32_t *>(&a);
            t.y = *reinterpret_cast<const uint32_t *>(&b);
            *reinterpret_cast<uint2 *>(static_cast<__half *>(y) + elem) = t;
        } else static_cast<__half *>(y)[elem] = __float2half_rn(v[0]);
    }
}

// S = stride, V = channels per thread (4 or 1), TX = output pixels per thread along x.
template <int DT, int S, int V, int TX>
__global__ void __launch_bounds__(256) dwconv_kernel(const DParams P) {
    constexpr int NC = (TX - 1) * S + 3;            // input columns a strip needs
    // blockIdx.x numbers groups of rows_per_block output rows (all images), blockIdx.y the
    // 256-thread pieces of a group's items; 32-bit arithmetic throughout.
    {
        const unsigned cv_n = (unsigned)(P.c / V);
        const unsigned local = blockIdx.y * blockDim.x + threadIdx.x;
        const unsigned row_local = local / (unsigned)P.items_per_row;
        if (row_local >= (unsigned)P.rows_per_block) return;
        const unsigned rem = local - row_local * (unsigned)P.items_per_row;
        const unsigned row = blockIdx.x * (unsigned)P.rows_per_block + row_local;
        if (row >= (unsigned)P.rows) return;
        const int strip = (int)(rem / cv_n);
        const int cv = (int)(rem - (unsigned)strip * cv_n);
        const int n = (int)(row / (unsigned)P.ho);
        const int oy = (int)(row - (unsigned)n * (unsigned)P.ho);
        const int ch = cv * V;
        const int ox0 = strip * TX;
        float acc[TX][V];
#pragma unroll
        for (int t = 0; t < TX; ++t)
#pragma unroll
            for (int v = 0; v < V; ++v) acc[t][v] = 0.0f;
        // Tensors hold fewer than 2^31 elements, so element offsets are 32-bit.  Which of the strip's
        // input columns lie inside the image is the same for the three rows: decided once.
        unsigned col_off[NC];
        bool col_ok[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) {
            const int ix = ox0 * S + j - 1;
            col_ok[j] = ix >= 0 && ix < P.w;
            col_off[j] = (unsigned)(col_ok[j] ? ix : 0) * (unsigned)P.c + (unsigned)ch;
        }
        // one input row at a time (holding all three rows in registers at once measured slower:
        // fewer threads fit an SM)
#pragma unroll
        for (int dy = 0; dy < 3; ++dy) {
            const int iy = oy * S + dy - 1;
            if (iy < 0 || iy >= P.h) continue;
            float wt[3][V];
#pragma unroll
            for (int dx = 0; dx < 3; ++dx) load_vec<XGEN_F32, V>(P.w9, (unsigned)(3 * dy + dx) * (unsigned)P.c + (unsigned)ch, wt[dx]);
            float col[NC][V];
            const unsigned row = ((unsigned)n * (unsigned)P.h + (unsigned)iy) * (unsigned)P.w * (unsigned)P.c;
#pragma unroll
            for (int j = 0; j < NC; ++j) {
                if (col_ok[j]) load_vec<DT, V>(P.x, row + col_off[j], col[j]);
                else {
#pragma unroll
                    for (int v = 0; v < V; ++v) col[j][v] = 0.0f;
                }
            }
#pragma unroll
            for (int t = 0; t < TX; ++t)
#pragma unroll
                for (int dx = 0; dx < 3; ++dx)
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[t][v] = fmaf(wt[dx][v], col[t * S + dx][v], acc[t][v]);
        }
        float b[V];
        if (P.bias) load_vec<XGEN_F32, V>(P.bias, (unsigned)ch, b);
        else {
#pragma unroll
            for (int v = 0; v < V; ++v) b[v] = 0.0f;
        }
#pragma unroll
        for (int t = 0; t < TX; ++t) {
            const int ox = ox0 + t;
            if (ox >= P.wo) break;
            float o[V];
#pragma unroll
            for (int v = 0; v < V; ++v) {
                o[v] = acc[t][v] + b[v];
                if (P.relu) o[v] = fmaxf(o[v], 0.0f);
            }
            store_vec<DT, V>(P.y, (((unsigned)n * (unsigned)P.ho + (unsigned)oy) * (unsigned)P.wo + (unsigned)ox) * (unsigned)P.c + (unsigned)ch, o);
        }
    }
}

constexpr int kStrip1 = 4, kStrip2 = 2;     // output pixels per thread at stride 1 / 2

static const void *kernel_for(xgen_dtype dt, int stride, bool vec) {
    if (dt == XGEN_F32) {
        if (stride == 1) return vec ? (const void *)dwconv_kernel<XGEN_F32, 1, 4, kStrip1> : (const void *)dwconv_kernel<XGEN_F32, 1, 1, kStrip1>;
        return vec ? (const void *)dwconv_kernel<XGEN_F32, 2, 4, kStrip2> : (const void *)dwconv_kernel<XGEN_F32, 2, 1, kStrip2>;
    }
    if (stride == 1) return vec ? (const void *)dwconv_kernel<XGEN_F16_F32ACC, 1, 4, kStrip1> : (const void *)dwconv_kernel<XGEN_F16_F32ACC, 1, 1, kStrip1>;
    return vec ? (const void *)dwconv_kernel<XGEN_F16_F32ACC, 2, 4, kStrip2> : (const void *)dwconv_kernel<XGEN_F16_F32ACC, 2, 1, kStrip2>;
}

static float half_bits_to_float(uint16_t h) {
    const uint32_t sign = (uint32_t)(h >> 15) << 31;
    const int exp = (h >> 10) & 0x1f;
    uint32_t man = h & 0x3ff, bits;
    if (exp == 0) {
        if (man == 0) bits = sign;
        else {
            int e = -1;
            do { ++e; man <<= 1; } while (!(man & 0x400));
            bits = sign | (uint32_t)(127 - 15 - e) << 23 | (man & 0x3ff) << 13;
        }
    } else if (exp == 31) bits = sign | 0x7f800000u | man << 13;
    else bits = sign | (uint32_t)(exp - 15 + 127) << 23 | man << 13;
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

}  // namespace dwconv

using namespace dwconv;

extern "C" {

xgen_status xgen_dwconv_pack(const xgen_dwconv_desc *d, const void *dense_w, const int16_t *pid, int device,
                             xgen_dwconv_packed **out) {
    if (!d || !dense_w || !pid || !out || !d->pattern_masks) return XGEN_ERR_INVALID_ARG;
    *out = nullptr;
    if (d->channels < 1) return XGEN_ERR_INVALID_ARG;
    if (d->pad != 1 || (d->stride != 1 && d->stride != 2)) return XGEN_ERR_UNSUPPORTED;
    if (d->dtype != XGEN_F32 && d->dtype != XGEN_F16_F32ACC) return XGEN_ERR_UNSUPPORTED;
    if (d->num_patterns < 1 || d->num_patterns > patconv::kNumAllMasks) return XGEN_ERR_BAD_PATTERN;
    for (int p = 0; p < d->num_patterns; ++p) {
        const uint16_t m = d->pattern_masks[p];
        if (m >= 512 || __builtin_popcount(m) != 4) return XGEN_ERR_BAD_PATTERN;
    }
    xgen_dwconv_packed *h = new (std::nothrow) xgen_dwconv_packed();
    if (!h) return XGEN_ERR_ALLOC;
    try {
        h->c = d->channels; h->stride = d->stride; h->dtype = d->dtype; h->device = device;
        h->w9.assign((size_t)9 * d->channels, 0.0f);
        for (int c = 0; c < d->channels; ++c) {
            const int p = pid[c];
            if (p >= d->num_patterns || p < -1) { delete h; return XGEN_ERR_BAD_PATTERN; }
            if (p < 0) continue;
            ++h->surviving;
            for (int t = 0; t < 9; ++t) {
                if (!((d->pattern_masks[p] >> t) & 1)) continue;
                const size_t i = (size_t)c * 9 + t;
                h->w9[(size_t)t * d->channels + c] = d->dtype == XGEN_F32 ? static_cast<const float *>(dense_w)[i]
                                                                           : half_bits_to_float(static_cast<const uint16_t *>(dense_w)[i]);
            }
        }
    } catch (const std::bad_alloc &) {
        delete h;
        return XGEN_ERR_ALLOC;
    }
    if (device >= 0) {
        int prev = 0;
        cudaGetDevice(&prev);
        xgen_status st = XGEN_OK;
        if (cudaSetDevice(device) != cudaSuccess) st = XGEN_ERR_CUDA;
        if (st == XGEN_OK && cudaMalloc(&h->d_w9, h->w9.size() * 4) != cudaSuccess) st = XGEN_ERR_ALLOC;
        if (st == XGEN_OK && cudaMemcpy(h->d_w9, h->w9.data(), h->w9.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) st = XGEN_ERR_CUDA;
        cudaSetDevice(prev);
        if (st != XGEN_OK) {
            cudaGetLastError();
            xgen_dwconv_free(h);
            return st;
        }
    }
    *out = h;
    return XGEN_OK;
}

xgen_status xgen_dwconv_run(const xgen_dwconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                            const void *bias, int32_t relu, void *y, void *stream) {
    if (!h || !x || !y) return XGEN_ERR_INVALID_ARG;
    const size_t eb = h->dtype == XGEN_F32 ? 4 : 2;
    if (((uintptr_t)x % eb) || ((uintptr_t)y % eb) || ((uintptr_t)bias % 4)) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    const int ho = (hh + 2 - 3) / h->stride + 1, wo = (ww + 2 - 3) / h->stride + 1;
    const int64_t xe = (int64_t)n * hh * ww * h->c, ye = (int64_t)n * ho * wo * h->c;
    if (xe > 2147483647LL || ye > 2147483647LL) return XGEN_ERR_SHAPE;
    {
        const uintptr_t xa = (uintptr_t)x, xz = xa + (size_t)xe * eb, ya = (uintptr_t)y, yz = ya + (size_t)ye * eb;
        if (xa < yz && ya < xz) return XGEN_ERR_INVALID_ARG;
    }
    if (h->device < 0) return XGEN_ERR_CUDA;
    const size_t vb = 4 * eb;                                   // bytes of four channels
    const bool vec = h->c % 4 == 0 && (uintptr_t)x % vb == 0 && (uintptr_t)y % vb == 0 && (uintptr_t)bias % 16 == 0;
    const int tx = h->stride == 1 ? kStrip1 : kStrip2;
    DParams P{};
    P.x = x; P.y = y; P.bias = static_cast<const float *>(bias); P.w9 = h->d_w9;
    P.n = n; P.h = hh; P.w = ww; P.ho = ho; P.wo = wo; P.c = h->c;
    P.relu = relu ? 1 : 0;
    P.strips = (wo + tx - 1) / tx;
    P.items_per_row = P.strips * (h->c / (vec ? 4 : 1));
    P.rows = n * ho;
    P.rows_per_block = std::max(1, std::min(256 / P.items_per_row, P.rows));
    int prev = 0;
    cudaGetDevice(&prev);
    if (prev != h->device && cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    const unsigned gx = (unsigned)((P.rows + P.rows_per_block - 1) / P.rows_per_block);
    const unsigned gy = (unsigned)(((long long)P.items_per_row * P.rows_per_block + 255) / 256);
    if (gy > 65535u) { if (prev != h->device) cudaSetDevice(prev); return XGEN_ERR_SHAPE; }
    void *args[] = {&P};
    xgen_status st = XGEN_OK;
    if (cudaLaunchKernel(kernel_for(h->dtype, h->stride, vec), dim3(gx, gy), dim3(256), args, 0, (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        st = XGEN_ERR_CUDA;
    } else patconv::count_launch();
    if (prev != h->device) cudaSetDevice(prev);
    return st;
}

xgen_status xgen_dwconv_query(const xgen_dwconv_packed *h, int64_t *kernels_surviving) {
    if (!h || !kernels_surviving) return XGEN_ERR_INVALID_ARG;
    *kernels_surviving = h->surviving;
    return XGEN_OK;
}

void xgen_dwconv_free(xgen_dwconv_packed *h) {
    if (!h) return;
    if (h->device >= 0 && h->d_w9) {
        int prev = 0;
        cudaGetDevice(&prev);
        if (cudaSetDevice(h->device) == cudaSuccess) cudaFree(h->d_w9);
        cudaSetDevice(prev);
    }
    delete h;
}

}  // extern "C"
