// Eq. 15-16: scatter the layer output back to the full token map, fill the pruned rows from
// the previous scale's residual cache (bilinear resize, half-pixel centres) and write the new
// residual cache.
//
// One warp per output row, 128-bit loads and stores. Work item r < M is kept row r of the
// compacted output; work item r >= M is entry r - M of the pruned index list. Every byte of
// x_in, y_kept, x_out and cache_out is touched exactly once; cache_prev is small and re-read
// through L2.
#include "common.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ uint4 ld_nc(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_cs(uint4* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void unpack2(uint32_t w, float& lo, float& hi)
{
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
restore_kernel(const uint4* __restrict__ x_in, const uint4* __restrict__ y_kept,
               const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ prune_idx,
               const int32_t* __restrict__ cu_keep, const uint4* __restrict__ cache_prev,
               int hp, int wp, int h, int w, int vec_per_row, int B, int M, bool m_on_device, bool pruned_only,
               uint4* __restrict__ x_out, uint4* __restrict__ cache_out)
{
    if (m_on_device) M = cu_keep[B];    // the kept count lives on the device
    const int lane = threadIdx.x & 31;
    // pruned_only: the kept rows were already written (by the block's last epilogue); work items
    // start at the first pruned entry
    const long r = (long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5) + (pruned_only ? M : 0);
    const int N = h * w;
    const long total = (long)B * N;
    if (r >= total) return;

    if (r < M) {
        // kept row: find its image (largest b with cu_keep[b] <= r)
        int lo = 0, hi = B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (cu_keep[mid] <= r) lo = mid; else hi = mid;
        }
        const long row = (long)lo * N + keep_idx[r];
        const uint4* ysrc = y_kept + r * vec_per_row;
        const uint4* xsrc = x_in + row * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32) {
            const uint4 yv = ld_nc(ysrc + v);
            st_cs(x_out + row * vec_per_row + v, yv);
            if (cache_out) {
                const uint4 xv = ld_nc(xsrc + v);
                const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w}, xw[4] = {xv.x, xv.y, xv.z, xv.w};
                uint32_t o[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float y0, y1, x0, x1;
                    unpack2(yw[q], y0, y1);
                    unpack2(xw[q], x0, x1);
                    o[q] = pack2(y0 - x0, y1 - x1);
                }
                st_cs(cache_out + row * vec_per_row + v, make_uint4(o[0], o[1], o[2], o[3]));
            }
        }
        return;
    }

    // pruned row: entry p of the pruned list; image b has its entries at [b*N - cu_keep[b], ...)
    const long p = r - M;
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long)mid * N - cu_keep[mid] <= p) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int i = prune_idx[p];
    const int oy = i / w, ox = i - oy * w;
    float sy = ((float)oy + 0.5f) * ((float)hp / (float)h) - 0.5f;
    float sx = ((float)ox + 0.5f) * ((float)wp / (float)w) - 0.5f;
    sy = fmaxf(sy, 0.f);
    sx = fmaxf(sx, 0.f);
    int y0 = min((int)sy, hp - 1), x0 = min((int)sx, wp - 1);
    const int y1 = min(y0 + 1, hp - 1), x1 = min(x0 + 1, wp - 1);
    const float fy = sy - (float)y0, fx = sx - (float)x0;
    const float w00 = (1.f - fy) * (1.f - fx), w01 = (1.f - fy) * fx, w10 = fy * (1.f - fx), w11 = fy * fx;
    const uint4* c00 = cache_prev + (((long)b * hp + y0) * wp + x0) * vec_per_row;
    const uint4* c01 = cache_prev + (((long)b * hp + y0) * wp + x1) * vec_per_row;
    const uint4* c10 = cache_prev + (((long)b * hp + y1) * wp + x0) * vec_per_row;
    const uint4* c11 = cache_prev + (((long)b * hp + y1) * wp + x1) * vec_per_row;
    const long row = (long)b * N + i;
    for (int v = lane; v < vec_per_row; v += 32) {
        const uint4 xv = ld_nc(x_in + row * vec_per_row + v);
        const uint4 a = c00[v], bq = c01[v], c = c10[v], d = c11[v];
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bq.x, bq.y, bq.z, bq.w};
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, dw[4] = {d.x, d.y, d.z, d.w};
        uint32_t o[4], u[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float xl, xh, al, ah, bl, bh, cl, ch, dl, dh;
            unpack2(xw[q], xl, xh);
            unpack2(aw[q], al, ah);
            unpack2(bw[q], bl, bh);
            unpack2(cw[q], cl, ch);
            unpack2(dw[q], dl, dh);
            const float ul = w00 * al + w01 * bl + w10 * cl + w11 * dl;
            const float uh = w00 * ah + w01 * bh + w10 * ch + w11 * dh;
            u[q] = pack2(ul, uh);
            o[q] = pack2(xl + ul, xh + uh);
        }
        st_cs(x_out + row * vec_per_row + v, make_uint4(o[0], o[1], o[2], o[3]));
        if (cache_out) st_cs(cache_out + row * vec_per_row + v, make_uint4(u[0], u[1], u[2], u[3]));
    }
}

}  // namespace

static nova_status restore(nova_ctx* ctx, const void* x_in, const void* y_kept,
                           const int32_t* keep_idx, const int32_t* prune_idx,
                           const int32_t* cu_keep, const void* cache_prev,
                           int hp, int wp, int h, int w, int C, int B, int M, bool m_on_device,
                           void* x_out, void* cache_out, void* stream, bool pruned_only = false)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (B < 0 || h < 0 || w < 0 || C < 1 || M < 0 || (long)M > (long)B * h * w)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_restore_from_cache: bad sizes");
    const long total = (long)B * h * w;
    if (total == 0) return NOVA_OK;
    if (C % 8) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_restore_from_cache: C must be a multiple of 8");
    if (!x_in || !x_out || !cu_keep || (M > 0 && !pruned_only && (!y_kept || !keep_idx)))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_restore_from_cache: null pointer");
    if ((M < total || m_on_device) && (!prune_idx || !cache_prev || hp < 1 || wp < 1))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_restore_from_cache: pruned rows need prune_idx and cache_prev");
    if (x_out == x_in) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_restore_from_cache: x_out aliases x_in");
    if (!nova_aligned16(x_in) || !nova_aligned16(x_out) || !nova_aligned16(y_kept) ||
        !nova_aligned16(cache_prev) || !nova_aligned16(cache_out))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_restore_from_cache: tensors must be 16-byte aligned");
    NOVA_DEVICE_GUARD(ctx, "nova_restore_from_cache");
    {
        // pruned_only: the kept list is not read (and may be null)
        const nova_status chk = nova_debug_check_lists(ctx, "nova_restore_from_cache", pruned_only ? nullptr : keep_idx,
                                                       prune_idx, cu_keep, B, h * w, M, !m_on_device, (cudaStream_t)stream);
        if (chk != NOVA_OK) return chk;
    }
    // rows this launch may have to visit: all of them, or only the pruned ones (when the host knows M)
    const long items = (pruned_only && !m_on_device) ? total - M : total;
    if (items == 0) return NOVA_OK;
    const unsigned blocks = (unsigned)((items + kWarpsPerBlock - 1) / kWarpsPerBlock);
    nova_launch_scope scope(ctx, NOVA_K_RESTORE, (cudaStream_t)stream);
    restore_kernel<<<blocks, kWarpsPerBlock * 32, 0, (cudaStream_t)stream>>>(
        (const uint4*)x_in, (const uint4*)y_kept, keep_idx, prune_idx, cu_keep, (const uint4*)cache_prev,
        hp, wp, h, w, C / 8, B, M, m_on_device, pruned_only, (uint4*)x_out, (uint4*)cache_out);
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

extern "C" nova_status nova_restore_from_cache(nova_ctx* ctx, const void* x_in, const void* y_kept,
                                               const int32_t* keep_idx, const int32_t* prune_idx,
                                               const int32_t* cu_keep, const void* cache_prev,
                                               int hp, int wp, int h, int w, int C, int B, int M,
                                               void* x_out, void* cache_out, void* stream)
{
    return restore(ctx, x_in, y_kept, keep_idx, prune_idx, cu_keep, cache_prev, hp, wp, h, w, C, B, M, false,
                   x_out, cache_out, stream);
}

extern "C" nova_status nova_restore_from_cache_device(nova_ctx* ctx, const void* x_in, const void* y_kept,
                                                      const int32_t* keep_idx, const int32_t* prune_idx,
                                                      const int32_t* cu_keep, const void* cache_prev,
                                                      int hp, int wp, int h, int w, int C, int B,
                                                      void* x_out, void* cache_out, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    const long total = (long)B * h * w;
    if (total > 0x7fffffffL) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_restore_from_cache_device: too many rows");
    return restore(ctx, x_in, y_kept, keep_idx, prune_idx, cu_keep, cache_prev, hp, wp, h, w, C, B, (int)total, true,
                   x_out, cache_out, stream);
}


// Eq. 16 for the pruned rows only: used by nova_pruned_layer_forward, whose last GEMM epilogue has
// already written the kept rows of x_out and cache_out.
nova_status nova_restore_pruned_rows(nova_ctx* ctx, const void* x_in, const int32_t* prune_idx,
                                     const int32_t* cu_keep, const void* cache_prev,
                                     int hp, int wp, int h, int w, int C, int B, int M, bool m_on_device,
                                     void* x_out, void* cache_out, void* stream)
{
    return restore(ctx, x_in, nullptr, nullptr, prune_idx, cu_keep, cache_prev, hp, wp, h, w, C, B, M, m_on_device,
                   x_out, cache_out, stream, true);
}
