// CUDA-core kernels: the fp32 tiled GEMM, the generic (any shape / alignment) GEMM and
// convolution used when the tensor-core path's layout constraints do not hold, and the
// fixed-order split-K reduction.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tdx {

// Bounds-checked debug mode of the one-thread-per-output kernels (TDX_DEBUG_BOUNDS=1): every global index is compared
// with the extent of its operand first; an index outside it is NOT accessed -- the kernel records kStatusBounds in the
// device status word (reported by tdx_check_device_status as a definite error) and uses 0 instead.  Nothing traps.
enum : int { kStatusBounds = 8 };
struct BoundsCheck {
    int on;                          // 0: no checks (the normal build of the call)
    long long a_elems, b_elems, c_elems, r_elems;   // extents in elements: left operand / input, right operand / filter, output, residual
    int* status;
};
__device__ __forceinline__ bool in_bounds(const BoundsCheck& bc, long long i, long long extent) {
    if (!bc.on || (i >= 0 && i < extent)) return true;
    atomicCAS(bc.status, 0, kStatusBounds);
    return false;
}

__device__ __forceinline__ float ld_as_float(const float* p, long long i) { return __ldg(p + i); }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p, long long i) {
    return __bfloat162float(p[i]);
}
__device__ __forceinline__ float as_float(float v) { return v; }
__device__ __forceinline__ float as_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void st_from_float(float* p, long long i, float v) { p[i] = v; }
__device__ __forceinline__ void st_from_float(__nv_bfloat16* p, long long i, float v) {
    p[i] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------
// fp32 GEMM, C = beta * C + alpha * op(A) op(B): element (i,k) of op(A) at A[i*sa_i + k*sa_k], element (k,j) of
// op(B) at B[k*sb_k + j*sb_j]; the reduction runs k = 0..K-1 in order with fp32 FMAs; batch = blockIdx.z.
// For small problems: 32 x 32 tiles, 2 x 2 outputs per thread, and a 4-stage cp.async ring so that the
// global-load latency of K-tile t+3 hides behind the FMAs of tile t (a small problem has too few CTAs per SM
// to hide it any other way).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void cp_async_f32(float* smem_dst, const float* gmem_src, bool valid) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    const int src_bytes = valid ? 4 : 0;   // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__global__ void __launch_bounds__(256)
sgemm_small_kernel(int M, int N, int K, long long sa_i, long long sa_k, long long sb_k, long long sb_j, float alpha,
                   const float* __restrict__ A, const float* __restrict__ B, float* __restrict__ C, float beta = 0.0f,
                   long long batch_a = 0, long long batch_b = 0, long long batch_c = 0) {
    constexpr int BM = 32, BN = 32, BK = 32, ST = 4, LD = BM + 2;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // see sgemm_small_rowmajor_kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    A += blockIdx.z * batch_a;
    B += blockIdx.z * batch_b;
    C += blockIdx.z * batch_c;
    __shared__ __align__(16) float As[ST][BK][LD];
    __shared__ __align__(16) float Bs[ST][BK][LD];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;          // 16 x 16 threads, 2 x 2 outputs each
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ktiles = (K + BK - 1) / BK;

    auto load_tile = [&](int kt, int st) {
        const int k0 = kt * BK;
#pragma unroll
        for (int e = 0; e < (BM * BK) / 256; ++e) {
            const int idx = tid + e * 256;
            int i, k;
            if (sa_k == 1) { i = idx / BK; k = idx % BK; } else { i = idx % BM; k = idx / BM; }
            const int gi = m0 + i, gk = k0 + k;
            const bool ok = gi < M && gk < K;
            cp_async_f32(&As[st][k][i], A + (ok ? gi * sa_i + gk * sa_k : 0), ok);
        }
#pragma unroll
        for (int e = 0; e < (BN * BK) / 256; ++e) {
            const int idx = tid + e * 256;
            int j, k;
            if (sb_j == 1) { k = idx / BN; j = idx % BN; } else { j = idx / BK; k = idx % BK; }
            const int gj = n0 + j, gk = k0 + k;
            const bool ok = gj < N && gk < K;
            cp_async_f32(&Bs[st][k][j], B + (ok ? gk * sb_k + gj * sb_j : 0), ok);
        }
    };

    for (int s = 0; s < ST - 1; ++s) {
        if (s < ktiles) load_tile(s, s);
        cp_async_commit();
    }
    float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    for (int kt = 0; kt < ktiles; ++kt) {
        cp_async_wait<ST - 2>();
        __syncthreads();                               // tile kt has landed; everyone is done with tile kt-1
        if (kt + ST - 1 < ktiles) load_tile(kt + ST - 1, (kt + ST - 1) % ST);
        cp_async_commit();
        const int st = kt % ST;
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float2 a = *reinterpret_cast<const float2*>(&As[st][k][ty * 2]);
            const float2 b = *reinterpret_cast<const float2*>(&Bs[st][k][tx * 2]);
            acc[0][0] = fmaf(a.x, b.x, acc[0][0]);
            acc[0][1] = fmaf(a.x, b.y, acc[0][1]);
            acc[1][0] = fmaf(a.y, b.x, acc[1][0]);
            acc[1][1] = fmaf(a.y, b.y, acc[1][1]);
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int gi = m0 + ty * 2 + i;
        if (gi >= M) continue;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int gj = n0 + tx * 2 + j;
            if (gj < N) {
                float* c = C + static_cast<long long>(gi) * N + gj;
                *c = beta != 0.0f ? fmaf(beta, *c, alpha * acc[i][j]) : alpha * acc[i][j];
            }
        }
    }
}

// ---------------------------------------------------------------------------
// The same ring with larger tiles: BM x BN per CTA, TM x TN outputs per thread, ST stages of BK.  A TM x TN register
// tile needs (TM + TN) shared-memory reads for TM * TN FMAs (4 x 4: 2 FMAs per read, where the 2 x 2 tile of the
// small kernel has 1), so this is the kernel for problems that offer at least one 64 x 64 tile per SM.
// Same index maps, batch / beta handling and k-ascending fp32 FMA order as above.
// ---------------------------------------------------------------------------
template <int BM, int BN, int BK, int TM, int TN, int ST>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
sgemm_ring_kernel(int M, int N, int K, long long sa_i, long long sa_k, long long sb_k, long long sb_j, float alpha,
                  const float* __restrict__ A, const float* __restrict__ B, float* __restrict__ C, float beta,
                  long long batch_a, long long batch_b, long long batch_c) {
    constexpr int NT = (BM / TM) * (BN / TN);
    static_assert(TM == 4 && TN == 4, "register tile is read with one 16-byte load per operand");
    static_assert((BM * BK) % NT == 0 && (BN * BK) % NT == 0, "whole number of copies per thread");
    A += blockIdx.z * batch_a;
    B += blockIdx.z * batch_b;
    C += blockIdx.z * batch_c;
    __shared__ __align__(16) float As[ST][BK][BM + 4];
    __shared__ __align__(16) float Bs[ST][BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid % (BN / TN), ty = tid / (BN / TN);
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ktiles = (K + BK - 1) / BK;

    auto load_tile = [&](int kt, int st) {
        const int k0 = kt * BK;
#pragma unroll
        for (int e = 0; e < (BM * BK) / NT; ++e) {
            const int idx = tid + e * NT;
            int i, k;
            if (sa_k == 1) { i = idx / BK; k = idx % BK; } else { i = idx % BM; k = idx / BM; }
            const int gi = m0 + i, gk = k0 + k;
            const bool ok = gi < M && gk < K;
            cp_async_f32(&As[st][k][i], A + (ok ? gi * sa_i + gk * sa_k : 0), ok);
        }
#pragma unroll
        for (int e = 0; e < (BN * BK) / NT; ++e) {
            const int idx = tid + e * NT;
            int j, k;
            if (sb_j == 1) { k = idx / BN; j = idx % BN; } else { j = idx / BK; k = idx % BK; }
            const int gj = n0 + j, gk = k0 + k;
            const bool ok = gj < N && gk < K;
            cp_async_f32(&Bs[st][k][j], B + (ok ? gk * sb_k + gj * sb_j : 0), ok);
        }
    };

    for (int s = 0; s < ST - 1; ++s) {
        if (s < ktiles) load_tile(s, s);
        cp_async_commit();
    }
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;
    for (int kt = 0; kt < ktiles; ++kt) {
        cp_async_wait<ST - 2>();
        __syncthreads();                               // tile kt has landed; everyone is done with tile kt-1
        if (kt + ST - 1 < ktiles) load_tile(kt + ST - 1, (kt + ST - 1) % ST);
        cp_async_commit();
        const int st = kt % ST;
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[st][k][ty * TM]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[st][k][tx * TN]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int gi = m0 + ty * TM + i;
        if (gi >= M) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int gj = n0 + tx * TN + j;
            if (gj < N) {
                float* c = C + static_cast<long long>(gi) * N + gj;
                *c = beta != 0.0f ? fmaf(beta, *c, alpha * acc[i][j]) : alpha * acc[i][j];
            }
        }
    }
}

// Same tiling for the plain row-major case (A is M x K, B is K x N, K and N multiples of 4, 16-byte aligned
// bases): both operands move with 16-byte cp.async, A stays k-contiguous in shared memory.
__device__ __forceinline__ void cp_async_16(float* smem_dst, const float* gmem_src, bool valid) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    const int src_bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}

// What bounds a small problem on this kernel is not global memory but the shared-memory latency of the inner loop:
// with 2 x 2 outputs per thread every four FMAs wait for a shared-memory read, and a 32 x 32 tile offers only two
// warps per scheduler to hide it (256^3: 41 % issue utilisation, 9.7 k cycles per CTA).  So here the CTA's four groups
// of 64 threads each take one quarter of every 128-deep K tile, a thread owns 4 x 4 outputs (eight 16-byte reads per
// 64 FMAs), and the four partial tiles are added in a fixed order (group 0 + 1 + 2 + 3) through shared memory at the
// end: the result is deterministic, each group's chain runs k ascending.  Two K tiles of 128 are in flight ahead of the
// FMAs (three stages), which covers K <= 256 before the first FMA.
constexpr int kSmallBK = 128, kSmallStages = 3;
constexpr int kSmallLDA = kSmallBK + 4, kSmallLDB = 32 + 4;
constexpr int kSmallStageFloats = 32 * kSmallLDA + kSmallBK * kSmallLDB;
constexpr int kSmallRowmajorSmem = kSmallStages * kSmallStageFloats * 4;

__global__ void __launch_bounds__(256)
sgemm_small_rowmajor_kernel(int M, int N, int K, float alpha, const float* __restrict__ A, const float* __restrict__ B,
                            float* __restrict__ C) {
    constexpr int BM = 32, BN = 32, BK = kSmallBK, ST = kSmallStages, LDA = kSmallLDA, LDB = kSmallLDB;
    // launched with programmatic stream serialization: let the next kernel of the stream be scheduled, and touch
    // global memory only once the previous one has completed (no-ops for an ordinary launch)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ __align__(16) float ring[];
    const int tid = threadIdx.x;
    const int grp = tid >> 6;                         // which quarter of each K tile
    const int tx = tid & 7, ty = (tid & 63) >> 3;     // 8 x 8 threads per group; rows ty + 8 i, columns 4 tx + j
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ktiles = (K + BK - 1) / BK;

    auto load_tile = [&](int kt, int st) {
        const int k0 = kt * BK;
        float* as = ring + st * kSmallStageFloats;    // [m][k], 32 x 128
        float* bs = as + BM * LDA;                    // [k][n], 128 x 32
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = tid + e * 256;
            {
                const int row = idx >> 5, c4 = (idx & 31) * 4;
                const int gi = m0 + row, gk = k0 + c4;
                const bool ok = gi < M && gk < K;            // K % 4 == 0: a group is all in or all out
                cp_async_16(as + row * LDA + c4, A + (ok ? static_cast<long long>(gi) * K + gk : 0), ok);
            }
            {
                const int row = idx >> 3, c4 = (idx & 7) * 4;
                const int gk = k0 + row, gj = n0 + c4;
                const bool ok = gk < K && gj < N;
                cp_async_16(bs + row * LDB + c4, B + (ok ? static_cast<long long>(gk) * N + gj : 0), ok);
            }
        }
    };

    for (int s = 0; s < ST - 1; ++s) {
        if (s < ktiles) load_tile(s, s);
        cp_async_commit();
    }
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    for (int kt = 0; kt < ktiles; ++kt) {
        cp_async_wait<ST - 2>();
        __syncthreads();
        if (kt + ST - 1 < ktiles) load_tile(kt + ST - 1, (kt + ST - 1) % ST);
        cp_async_commit();
        const float* as = ring + (kt % ST) * kSmallStageFloats + ty * LDA + grp * 32;
        const float* bs = ring + (kt % ST) * kSmallStageFloats + BM * LDA + grp * 32 * LDB + tx * 4;
#pragma unroll
        for (int k4 = 0; k4 < 32; k4 += 4) {
            float a[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 v = *reinterpret_cast<const float4*>(as + i * 8 * LDA + k4);
                a[i][0] = v.x; a[i][1] = v.y; a[i][2] = v.z; a[i][3] = v.w;
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const float4 b = *reinterpret_cast<const float4*>(bs + (k4 + kk) * LDB);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[i][0] = fmaf(a[i][kk], b.x, acc[i][0]);
                    acc[i][1] = fmaf(a[i][kk], b.y, acc[i][1]);
                    acc[i][2] = fmaf(a[i][kk], b.z, acc[i][2]);
                    acc[i][3] = fmaf(a[i][kk], b.w, acc[i][3]);
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();                                   // every group is done with the ring: reuse it for the partial tiles
    constexpr int LDR = BN + 4;
    float* red = ring;                                 // [group][row][column]
#pragma unroll
    for (int i = 0; i < 4; ++i)
        *reinterpret_cast<float4*>(red + (grp * BM + ty + 8 * i) * LDR + tx * 4) =
            make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    __syncthreads();
    {
        const int row = tid >> 3, c4 = (tid & 7) * 4;   // 32 rows x 8 groups of 4 columns: one per thread
        float4 s = *reinterpret_cast<const float4*>(red + row * LDR + c4);
#pragma unroll
        for (int g = 1; g < 4; ++g) {
            const float4 v = *reinterpret_cast<const float4*>(red + (g * BM + row) * LDR + c4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        const int gi = m0 + row, gj = n0 + c4;
        if (gi < M && gj < N)                            // N % 4 == 0 and C 16-byte aligned: a group is all in or all out
            *reinterpret_cast<float4*>(C + static_cast<long long>(gi) * N + gj) =
                make_float4(alpha * s.x, alpha * s.y, alpha * s.z, alpha * s.w);
    }
}

// ---------------------------------------------------------------------------
// Generic GEMM, one thread per output element (no layout or alignment constraints).
// ---------------------------------------------------------------------------
template <typename TIn, typename TOut>
__global__ void gemm_generic_kernel(long long M, long long N, long long K, long long sa_i, long long sa_k,
                                    long long sb_k, long long sb_j, float alpha, const TIn* __restrict__ A,
                                    const TIn* __restrict__ B, TOut* __restrict__ C, float beta = 0.0f,
                                    long long batch = 1, long long batch_a = 0, long long batch_b = 0,
                                    long long batch_c = 0, BoundsCheck bc = BoundsCheck{0, 0, 0, 0, 0, nullptr}) {
    // batched: C[b] = beta * C[b] + alpha * A[b] . B[b]; C is not read when beta == 0
    const long long per = M * N, total = per * batch;
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < total;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long b = e / per, r = e - b * per;
        const long long i = r / N, j = r - i * N;
        float acc = 0.0f;
        if (bc.on) {
            // debug mode: indices relative to the operand's base, checked against its extent before every access
            for (long long k = 0; k < K; ++k) {
                const long long ia = b * batch_a + i * sa_i + k * sa_k, ib = b * batch_b + k * sb_k + j * sb_j;
                const float x = in_bounds(bc, ia, bc.a_elems) ? ld_as_float(A, ia) : 0.0f;
                const float y = in_bounds(bc, ib, bc.b_elems) ? ld_as_float(B, ib) : 0.0f;
                acc = fmaf(x, y, acc);
            }
            const long long ic = b * batch_c + r;
            if (!in_bounds(bc, ic, bc.c_elems)) continue;
        } else {
            const TIn* a = A + b * batch_a;
            const TIn* bb = B + b * batch_b;
            for (long long k = 0; k < K; ++k)
                acc = fmaf(ld_as_float(a, i * sa_i + k * sa_k), ld_as_float(bb, k * sb_k + j * sb_j), acc);
        }
        TOut* c = C + b * batch_c;
        float v = alpha * acc;
        if (beta != 0.0f) v = fmaf(beta, as_float(c[r]), v);     // plain load: this thread overwrites it next
        st_from_float(c, r, v);
    }
}

// ---------------------------------------------------------------------------
// Generic convolution + bias + ReLU, one thread per output element.  x NHWC, w KRSC.
// Taps that fall into the zero padding are skipped (they would add zero).
// ---------------------------------------------------------------------------
template <typename TIn, typename TOut>
__global__ void conv2d_generic_kernel(int Nimg, int H, int W, int Cin, int Cout, int R, int S, int pad, int stride,
                                      int P, int Q, const TIn* __restrict__ x, const TIn* __restrict__ w,
                                      const float* __restrict__ bias, int relu, TOut* __restrict__ y,
                                      const TOut* __restrict__ residual = nullptr,
                                      BoundsCheck bc = BoundsCheck{0, 0, 0, 0, 0, nullptr}) {
    const long long total = static_cast<long long>(Nimg) * P * Q * Cout;
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < total;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int k = static_cast<int>(e % Cout);
        long long row = e / Cout;
        const int q = static_cast<int>(row % Q);
        row /= Q;
        const int p = static_cast<int>(row % P);
        const int n = static_cast<int>(row / P);
        float acc = 0.0f;
        for (int r = 0; r < R; ++r) {
            const int h = p * stride + r - pad;
            if (h < 0 || h >= H) continue;
            for (int s = 0; s < S; ++s) {
                const int ww = q * stride + s - pad;
                if (ww < 0 || ww >= W) continue;
                const long long xo = ((static_cast<long long>(n) * H + h) * W + ww) * Cin;
                const long long wo = ((static_cast<long long>(k) * R + r) * S + s) * Cin;
                if (bc.on) {
                    for (int c = 0; c < Cin; ++c) {
                        const float xv = in_bounds(bc, xo + c, bc.a_elems) ? ld_as_float(x, xo + c) : 0.0f;
                        const float wv = in_bounds(bc, wo + c, bc.b_elems) ? ld_as_float(w, wo + c) : 0.0f;
                        acc = fmaf(xv, wv, acc);
                    }
                } else {
                    for (int c = 0; c < Cin; ++c) acc = fmaf(ld_as_float(x, xo + c), ld_as_float(w, wo + c), acc);
                }
            }
        }
        if (bias != nullptr) acc += __ldg(bias + k);
        if (residual != nullptr && in_bounds(bc, e, bc.r_elems)) acc += as_float(residual[e]);
        if (relu) acc = fmaxf(acc, 0.0f);
        if (!in_bounds(bc, e, bc.c_elems)) continue;
        st_from_float(y, e, acc);
    }
}

// ---------------------------------------------------------------------------
// Split-K reduction: out[i,j] = epilogue( sum_{s = 0..split-1, ascending} partial[s][i][j] ).
// The order is fixed, so results do not depend on scheduling.
// ---------------------------------------------------------------------------
// Batched (batch > 1): partial is [batch][split][MN] and batch b of out starts batch_c elements after batch b - 1.
__global__ void splitk_reduce_kernel(long long MN, int N, int split, const float* __restrict__ partial, float alpha,
                                     const float* __restrict__ bias, int relu, __nv_bfloat16* __restrict__ out,
                                     int vec8, float beta = 0.0f, int batch = 1, long long batch_c = 0) {
    // launched with programmatic stream serialization: this grid may start while the GEMM drains; wait here
    // until the GEMM grid has completed and its partial sums are visible (a no-op for an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (batch > 1) {
        // one element (or one group of eight) per thread and pass, batches included; same fixed order of the splits
        const long long per = vec8 ? MN / 8 : MN, total = per * batch;
        for (long long gg = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; gg < total;
             gg += static_cast<long long>(gridDim.x) * blockDim.x) {
            const long long b = gg / per, g = gg - b * per;
            const float* pb = partial + b * split * MN;
            __nv_bfloat16* ob = out + b * batch_c;
            if (vec8) {
                const long long e = g * 8;
                float acc[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
                uint4 old = make_uint4(0u, 0u, 0u, 0u);
                if (beta != 0.0f) old = *reinterpret_cast<const uint4*>(ob + e);
#pragma unroll 4
                for (int s = 0; s < split; ++s) {
                    const float4* src = reinterpret_cast<const float4*>(pb + s * MN + e);
                    const float4 v0 = __ldg(src), v1 = __ldg(src + 1);
                    acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
                    acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
                }
                const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
                uint32_t pk[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float a = alpha * acc[2 * j], c = alpha * acc[2 * j + 1];
                    if (beta != 0.0f) {
                        a = fmaf(beta, __uint_as_float(ow[j] << 16), a);
                        c = fmaf(beta, __uint_as_float(ow[j] & 0xFFFF0000u), c);
                    }
                    __nv_bfloat162 h = __floats2bfloat162_rn(a, c);
                    pk[j] = *reinterpret_cast<uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(ob + e) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            } else {
                float acc = 0.0f;
                for (int s = 0; s < split; ++s) acc += __ldg(pb + s * MN + g);
                float v = alpha * acc;
                if (beta != 0.0f) v = fmaf(beta, __bfloat162float(ob[g]), v);
                ob[g] = __float2bfloat16_rn(v);
            }
        }
        return;
    }
    if (vec8) {
        const long long groups = MN / 8;
        for (long long g = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; g < groups;
             g += static_cast<long long>(gridDim.x) * blockDim.x) {
            const long long e = g * 8;
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
            // unrolled so that the loads of four splits are in flight together (the adds keep their order)
#pragma unroll 4
            for (int s = 0; s < split; ++s) {
                const float4* src = reinterpret_cast<const float4*>(partial + s * MN + e);
                const float4 v0 = __ldg(src), v1 = __ldg(src + 1);
                acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
                acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
            }
            const int col = static_cast<int>(e % N);
            uint32_t pk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float a = alpha * acc[2 * j], b = alpha * acc[2 * j + 1];
                if (beta != 0.0f) {          // accumulate into what the output held
                    a = fmaf(beta, __bfloat162float(out[e + 2 * j]), a);
                    b = fmaf(beta, __bfloat162float(out[e + 2 * j + 1]), b);
                }
                if (bias != nullptr) { a += __ldg(bias + col + 2 * j); b += __ldg(bias + col + 2 * j + 1); }
                if (relu) { a = fmaxf(a, 0.0f); b = fmaxf(b, 0.0f); }
                __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                pk[j] = *reinterpret_cast<uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(out + e) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    } else {
        for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < MN;
             e += static_cast<long long>(gridDim.x) * blockDim.x) {
            float acc = 0.0f;
            for (int s = 0; s < split; ++s) acc += __ldg(partial + s * MN + e);
            float v = alpha * acc;
            if (beta != 0.0f) v = fmaf(beta, __bfloat162float(out[e]), v);
            if (bias != nullptr) v += __ldg(bias + e % N);
            if (relu) v = fmaxf(v, 0.0f);
            out[e] = __float2bfloat16_rn(v);
        }
    }
}

// The same reduction for the K-balanced plan, where the number of partial tiles differs from tile to tile:
// nseg[row block * tiles_n + column tile] slots hold that tile's partial sums (slot s at partial + s * MN), added in
// ascending slot order = ascending K.  Tiles are bm rows x bn columns (bn a multiple of 8).
__global__ void splitk_reduce_var_kernel(long long MN, int N, int bm, int bn, int tiles_n, const int* __restrict__ nseg,
                                         const float* __restrict__ partial, float alpha, __nv_bfloat16* __restrict__ out,
                                         int vec8, float beta) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long per = vec8 ? MN / 8 : MN;
    for (long long g = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; g < per;
         g += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long e = vec8 ? g * 8 : g;
        const long long row = e / N;
        const int col = static_cast<int>(e - row * N);
        const int split = __ldg(nseg + (row / bm) * tiles_n + col / bn);
        if (vec8) {
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
#pragma unroll 4
            for (int s = 0; s < split; ++s) {
                const float4* src = reinterpret_cast<const float4*>(partial + s * MN + e);
                const float4 v0 = __ldg(src), v1 = __ldg(src + 1);
                acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
                acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
            }
            uint32_t pk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float a = alpha * acc[2 * j], b = alpha * acc[2 * j + 1];
                if (beta != 0.0f) {
                    a = fmaf(beta, __bfloat162float(out[e + 2 * j]), a);
                    b = fmaf(beta, __bfloat162float(out[e + 2 * j + 1]), b);
                }
                __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                pk[j] = *reinterpret_cast<uint32_t*>(&h);
            }
            *reinterpret_cast<uint4*>(out + e) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        } else {
            float acc = 0.0f;
            for (int s = 0; s < split; ++s) acc += __ldg(partial + s * MN + e);
            float v = alpha * acc;
            if (beta != 0.0f) v = fmaf(beta, __bfloat162float(out[e]), v);
            out[e] = __float2bfloat16_rn(v);
        }
    }
}

// ---------------------------------------------------------------------------
// add(zero_pad(x), y) without the padded copy and without adding the zeros: out = y, plus x inside the interior.
// x is N x H x W x C, y / out are N x Hp x Wp x C.  An interior row (n, h) is W * C contiguous elements in x and
// in y.  In place (out == y) only the interior is read and written: the padding ring is never touched.  Out of
// place the ring is copied.  `vec` = elements per 16-byte access when every row start is 16-byte aligned, else 1.
// HBM-bound: 3 x interior bytes in place.
// ---------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void add_vec16(const T* __restrict__ a, const T* b, T* o) {
    constexpr int V = 16 / sizeof(T);
    const uint4 ua = __ldg(reinterpret_cast<const uint4*>(a));
    const uint4 ub = *reinterpret_cast<const uint4*>(b);
    const T* pa = reinterpret_cast<const T*>(&ua);
    const T* pb = reinterpret_cast<const T*>(&ub);
    uint4 uo;
    T* po = reinterpret_cast<T*>(&uo);
#pragma unroll
    for (int i = 0; i < V; ++i) st_from_float(po, i, as_float(pa[i]) + as_float(pb[i]));
    *reinterpret_cast<uint4*>(o) = uo;
}

template <typename T>
__global__ void add_zero_pad_kernel(long long rows, long long H, long long row_elems, long long y_img_elems,
                                    long long y_row_elems, long long y_first, int vec, const T* __restrict__ x,
                                    const T* y, T* out) {
    // row r = (n, h): x + r * row_elems  <->  y + n * y_img_elems + y_first + h * y_row_elems
    // launched with programmatic stream serialization (see sgemm_small_rowmajor_kernel)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long per_row = vec > 1 ? row_elems / vec : row_elems;
    const long long total = rows * per_row;
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < total;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long r = e / per_row, i = (e - r * per_row) * (vec > 1 ? vec : 1);
        const long long n = r / H, h = r - n * H;
        const long long xo = r * row_elems + i;
        const long long yo = n * y_img_elems + y_first + h * y_row_elems + i;
        if (vec > 1) add_vec16<T>(x + xo, y + yo, out + yo);
        else st_from_float(out, yo, as_float(x[xo]) + as_float(y[yo]));
    }
}

// out-of-place only: copies the elements of y outside the interior (the padding ring) to out
template <typename T>
__global__ void copy_pad_ring_kernel(long long total, long long C, long long Hp, long long Wp, long long top, long long H,
                                     long long left, long long W, const T* __restrict__ y, T* __restrict__ out) {
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < total;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long pix = e / C;
        const long long w = pix % Wp, h = (pix / Wp) % Hp;
        if (h < top || h >= top + H || w < left || w >= left + W) out[e] = y[e];
    }
}

// The same reduction with an fp32 result: out = alpha * sum_s partial[s] + beta * out (the fp32 GEMM from bf16 pieces).
// Batched: partial is [batch][split][MN], batch b of out starts batch_c elements after batch b - 1.
__global__ void splitk_reduce_f32_kernel(long long MN, int split, const float* __restrict__ partial, float alpha, float beta,
                                         float* out, int vec4, int batch = 1, long long batch_c = 0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (vec4) {
        const long long per = MN / 4, groups = per * batch;
        for (long long gg = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; gg < groups;
             gg += static_cast<long long>(gridDim.x) * blockDim.x) {
            const long long b = gg / per, g = gg - b * per;
            const float* pb = partial + b * split * MN;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            // the accumulate term is fetched before the partial sums are needed, and the loads of several splits
            // are in flight together (the adds keep their order)
            float4 old = make_float4(0.f, 0.f, 0.f, 0.f);
            if (beta != 0.0f) old = *(reinterpret_cast<const float4*>(out + b * batch_c) + g);
#pragma unroll 8
            for (int s = 0; s < split; ++s) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(pb + s * MN) + g);
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            float4 r = make_float4(alpha * acc.x, alpha * acc.y, alpha * acc.z, alpha * acc.w);
            float4* o = reinterpret_cast<float4*>(out + b * batch_c) + g;
            if (beta != 0.0f) {
                r.x = fmaf(beta, old.x, r.x); r.y = fmaf(beta, old.y, r.y); r.z = fmaf(beta, old.z, r.z); r.w = fmaf(beta, old.w, r.w);
            }
            *o = r;
        }
    } else {
        for (long long ee = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; ee < MN * batch;
             ee += static_cast<long long>(gridDim.x) * blockDim.x) {
            const long long b = ee / MN, e = ee - b * MN;
            float acc = 0.0f;
            for (int s = 0; s < split; ++s) acc += __ldg(partial + (b * split + s) * MN + e);
            const float v = alpha * acc;
            float* o = out + b * batch_c + e;
            *o = beta != 0.0f ? fmaf(beta, *o, v) : v;
        }
    }
}

// ---------------------------------------------------------------------------
// fp32 -> three bf16 pieces, for the fp32 GEMM on the tensor cores: x = hi + mid + lo with hi = bf16(x),
// mid = bf16(x - hi), lo = bf16(x - hi - mid); both differences are exact in fp32 and the three pieces carry all
// 24 significand bits.  Source: `rows` x K logical matrix, element (i, k) at src[b * batch_stride + i * s_row + k * s_k]
// (either stride may be 1).  Destination, per batch: rows x (3 * Kp) bf16, row-major, piece p of element (i, k) at
// column p * Kp + k; columns K..Kp-1 of every piece are zero (Kp is K rounded up to the K block of the MMA pipeline).
// Tiles of 32 rows x 64 columns through shared memory, so that reads and writes are both coalesced whichever stride
// is 1; a thread issues its eight loads back to back and writes pairs of pieces (4-byte stores, whole 128-byte lines
// per warp).
// ---------------------------------------------------------------------------
// One launch may split two operands (A and B of a GEMM): blockIdx.z below `nb0` works on the first, the rest on the
// second; an operand with fewer 32-row blocks than the grid has lets the surplus CTAs leave at once.
struct SplitOperand {
    int rows;
    long long s_row, s_k, batch_stride;
    const float* src;
    __nv_bfloat16* dst;
};
__global__ void __launch_bounds__(256)
split_f32_bf16x3_kernel(int K, int Kp, int nb0, SplitOperand op0, SplitOperand op1) {
    __shared__ float tile[32][65];
    const bool second = static_cast<int>(blockIdx.z) >= nb0;
    const SplitOperand& op = second ? op1 : op0;
    const int rows = op.rows;
    const long long s_row = op.s_row, s_k = op.s_k;
    const int bz = static_cast<int>(blockIdx.z) - (second ? nb0 : 0);
    // launched with programmatic stream serialization (see sgemm_small_rowmajor_kernel): the piece buffers are shared
    // by successive calls, and the wait orders this kernel after everything the stream held before it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int k0 = blockIdx.x * 64, r0 = blockIdx.y * 32;
    if (r0 >= rows) return;                           // CTA-uniform: before any barrier
    const float* s = op.src + bz * op.batch_stride;
    __nv_bfloat16* d = op.dst + static_cast<long long>(bz) * rows * 3 * Kp;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;        // 32 x 8 threads
    if (s_k == 1) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int jj = ty + 8 * j, r = r0 + jj;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int k = k0 + tx + 32 * h;
                tile[jj][tx + 32 * h] = (r < rows && k < K) ? __ldg(s + r * s_row + k) : 0.0f;
            }
        }
    } else {       // rows are the contiguous dimension of the source: read along them, transpose in shared memory
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int kk = ty + 8 * j, k = k0 + kk, r = r0 + tx;
            tile[tx][kk] = (r < rows && k < K) ? __ldg(s + r * s_row + k * s_k) : 0.0f;
        }
    }
    __syncthreads();
    const int k = k0 + 2 * tx;                                     // Kp is a multiple of 64: a pair is all in or all out
    if (k < Kp) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int jj = ty + 8 * j, r = r0 + jj;
            if (r >= rows) continue;
            const float x0 = tile[jj][2 * tx], x1 = tile[jj][2 * tx + 1];
            const __nv_bfloat162 hi = __floats2bfloat162_rn(x0, x1);
            const float r0x = x0 - __low2float(hi), r1x = x1 - __high2float(hi);
            const __nv_bfloat162 mid = __floats2bfloat162_rn(r0x, r1x);
            const __nv_bfloat162 lo = __floats2bfloat162_rn(r0x - __low2float(mid), r1x - __high2float(mid));
            __nv_bfloat16* o = d + static_cast<long long>(r) * 3 * Kp + k;
            *reinterpret_cast<__nv_bfloat162*>(o) = hi;
            *reinterpret_cast<__nv_bfloat162*>(o + Kp) = mid;
            *reinterpret_cast<__nv_bfloat162*>(o + 2 * Kp) = lo;
        }
    }
}

// ---------------------------------------------------------------------------
// bf16 operand -> K-major copy with K padded to the MMA pipeline's K block: for operands whose layout the copy
// engine cannot address (a row pitch that is no multiple of 16 bytes -- K = 2305 is the paper's own example -- or a
// misaligned base).  Source: `rows` x K logical matrix, element (i, k) at src[b * batch_stride + i * s_row + k * s_k]
// (either stride may be 1).  Destination, per batch: rows x Kp bf16, row-major, columns K..Kp-1 zero.  The padding
// adds exact zeros to every sum, so the result is that of the unpadded reduction.  Same tiling as the fp32 piece
// kernel below: 32 rows x 64 columns through shared memory, both operands of a GEMM in one launch.
// ---------------------------------------------------------------------------
struct PadOperand {
    int rows;
    long long s_row, s_k, batch_stride;
    const __nv_bfloat16* src;
    __nv_bfloat16* dst;
};
__global__ void __launch_bounds__(256)
pad_k_bf16_kernel(int K, int Kp, int nb0, PadOperand op0, PadOperand op1) {
    __shared__ __nv_bfloat16 tile[32][66];
    const bool second = static_cast<int>(blockIdx.z) >= nb0;
    const PadOperand& op = second ? op1 : op0;
    const int rows = op.rows;
    const long long s_row = op.s_row, s_k = op.s_k;
    const int bz = static_cast<int>(blockIdx.z) - (second ? nb0 : 0);
    // launched with programmatic stream serialization: the scratch copies are shared by successive calls, and the
    // wait orders this kernel after everything the stream held before it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int k0 = blockIdx.x * 64, r0 = blockIdx.y * 32;
    if (r0 >= rows) return;                           // CTA-uniform: before any barrier
    const __nv_bfloat16* s = op.src + bz * op.batch_stride;
    __nv_bfloat16* d = op.dst + static_cast<long long>(bz) * rows * Kp;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;        // 32 x 8 threads
    const __nv_bfloat16 zero = __float2bfloat16_rn(0.0f);
    if (s_k == 1) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int jj = ty + 8 * j, r = r0 + jj;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int k = k0 + tx + 32 * h;
                tile[jj][tx + 32 * h] = (r < rows && k < K) ? s[r * s_row + k] : zero;
            }
        }
    } else {       // rows are the contiguous dimension of the source: read along them, transpose in shared memory
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int kk = ty + 8 * j, k = k0 + kk, r = r0 + tx;
            tile[tx][kk] = (r < rows && k < K) ? s[r * s_row + k * s_k] : zero;
        }
    }
    __syncthreads();
    const int k = k0 + 2 * tx;                                     // Kp is a multiple of 64: a pair is all in or all out
    if (k < Kp) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int jj = ty + 8 * j, r = r0 + jj;
            if (r >= rows) continue;
            __nv_bfloat162 v;
            v.x = tile[jj][2 * tx];
            v.y = tile[jj][2 * tx + 1];
            *reinterpret_cast<__nv_bfloat162*>(d + static_cast<long long>(r) * Kp + k) = v;
        }
    }
}

// max |a - b| and max |b| over n bf16 values -> out[0], out[1] as fp32 bit patterns (non-negative floats order like
// unsigned integers, so atomicMax works on them; a NaN becomes +inf's pattern).  Used by the search to check a
// winner's output against the generic kernel's.
__global__ void max_diff_bf16_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ b, long long n,
                                     unsigned* out) {
    float d = 0.0f, m = 0.0f;
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < n;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const float x = __bfloat162float(a[e]), y = __bfloat162float(b[e]);
        float dd = fabsf(x - y), mm = fabsf(y);
        if (!(dd == dd)) dd = __int_as_float(0x7f800000);
        if (!(mm == mm)) mm = __int_as_float(0x7f800000);
        d = fmaxf(d, dd);
        m = fmaxf(m, mm);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        d = fmaxf(d, __shfl_xor_sync(0xffffffffu, d, o));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicMax(out, __float_as_uint(d));
        atomicMax(out + 1, __float_as_uint(m));
    }
}

// Deterministic pseudo-random fill used only by the tuner's scratch operands.
__global__ void fill_pattern_bf16_kernel(__nv_bfloat16* p, long long n, uint32_t seed) {
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < n;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        uint32_t h = static_cast<uint32_t>(e) * 2654435761u + seed;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        const float v = (static_cast<float>(h & 0xFFFF) - 32768.0f) * (1.0f / 16384.0f);
        p[e] = __float2bfloat16_rn(v);
    }
}

}  // namespace tdx
