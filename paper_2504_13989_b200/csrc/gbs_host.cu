// C-ABI entry points: argument validation, plan construction, kernel-family dispatch.
// Every argument error is caught here, on the host, before anything is launched.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "gbs_internal.h"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int log2_exact(int v)
{
    if (v < 1 || (v & (v - 1))) return -1;
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
}

bool supported_m(int m) { return gbs_supported_m(m); }

int elem_size(int dtype) { return dtype == GBS_DTYPE_F32 ? 4 : 2; }

// shared validation of (x, dtype, n_rows, stride)
int check_rows(const gbs_plan* p, const void* x, int x_dtype, int64_t n_rows, int64_t stride)
{
    if (!p) return GBS_ERR_INVALID_ARG;
    if (x_dtype != GBS_DTYPE_F32 && x_dtype != GBS_DTYPE_BF16) return GBS_ERR_INVALID_ARG;
    if (n_rows < 0) return GBS_ERR_INVALID_ARG;
    if (n_rows == 0) return GBS_OK;
    if (!x) return GBS_ERR_INVALID_ARG;
    if (stride < p->d) return GBS_ERR_INVALID_ARG;
    if (!aligned16(x) || ((stride * elem_size(x_dtype)) & 15) != 0) return GBS_ERR_ALIGNMENT;
    return GBS_OK;
}

typedef gbs_device_guard DeviceGuard;

}  // namespace

extern "C" int gbs_hadamard_m(int m, int8_t* out_host)
{
    if (!out_host || m < 1) return GBS_ERR_INVALID_ARG;
    if (!supported_m(m) && !gbs_supported_full_m(m)) return GBS_ERR_UNSUPPORTED;
    return gbs_build_hadamard_m(m, out_host);
}

extern "C" const char* gbs_status_string(int status)
{
    switch (status) {
        case GBS_OK: return "GBS_OK";
        case GBS_ERR_INVALID_ARG: return "GBS_ERR_INVALID_ARG: argument out of its documented range";
        case GBS_ERR_UNSUPPORTED: return "GBS_ERR_UNSUPPORTED: no Hadamard construction for this m, or d' too large";
        case GBS_ERR_ALIGNMENT: return "GBS_ERR_ALIGNMENT: pointer or stride not 16-byte aligned";
        case GBS_ERR_CUDA: return "GBS_ERR_CUDA: a CUDA runtime call failed";
        case GBS_ERR_ALLOC: return "GBS_ERR_ALLOC: allocation failed";
        default: return "GBS: unknown status";
    }
}

extern "C" int gbs_plan_create(gbs_plan_t** out, int d, int d_pad, int m, int bits, int group, float alpha)
{
    return gbs_plan_create_ex(out, d, d_pad, m, bits, group, alpha, 0);
}

extern "C" int gbs_plan_create_ex(gbs_plan_t** out, int d, int d_pad, int m, int bits, int group, float alpha,
                                  int flags)
{
    if (!out) return GBS_ERR_INVALID_ARG;
    if (flags & ~GBS_PLAN_ASYMMETRIC) return GBS_ERR_INVALID_ARG;
    if (d < 1 || d_pad < d || m < 1) return GBS_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4) return GBS_ERR_INVALID_ARG;
    if (!(alpha > 0.f) || !(alpha <= 1.f)) return GBS_ERR_INVALID_ARG;     // also rejects NaN
    if (d_pad % m != 0) return GBS_ERR_INVALID_ARG;
    const int k = log2_exact(d_pad / m);
    const bool full = (k == 0 && gbs_supported_full_m(m));                  // d' = m: the rotation is H_m itself
    if (k < 3 && !full) return GBS_ERR_INVALID_ARG;                         // 2^k >= 8
    if (group != 0) {
        if (group < 8 || log2_exact(group) < 0 || (1 << k) % group != 0) return GBS_ERR_INVALID_ARG;
    }
    if (!full && !supported_m(m)) return GBS_ERR_UNSUPPORTED;
    if (d_pad > GBS_MAX_D_PAD) return GBS_ERR_UNSUPPORTED;
    if (full && (group != 0 || (flags & GBS_PLAN_ASYMMETRIC) || d % 8 != 0)) return GBS_ERR_UNSUPPORTED;
    if ((flags & GBS_PLAN_ASYMMETRIC) &&
        !(d_pad == 128 && m == 1 && (group == 0 || group == 32 || group == 64 || group == 128)))
        return GBS_ERR_UNSUPPORTED;

    gbs_plan* p = new (std::nothrow) gbs_plan;
    if (!p) return GBS_ERR_ALLOC;
    memset(p, 0, sizeof(*p));
    p->d = d; p->d_pad = d_pad; p->m = m; p->k = k; p->bits = bits; p->group = group; p->alpha = alpha;
    p->levels = (1 << (bits - 1)) - 1;
    const double rootn = sqrt((double)d_pad);
    p->norm = (float)(1.0 / rootn);
    p->c_scale = (float)((double)alpha / ((double)p->levels * rootn));
    p->c_inv = (float)((double)p->levels / (double)alpha);
    p->variant = GBS_VARIANT_GENERIC;
    p->asym = (flags & GBS_PLAN_ASYMMETRIC) ? 1 : 0;
    int rc = full ? GBS_OK : gbs_build_hadamard_m(m, p->h_hm);          // a full order has no small factor to keep
    if (rc != GBS_OK) { delete p; return rc; }

    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device);
    if (e != cudaSuccess) { cudaGetLastError(); delete p; return GBS_ERR_CUDA; }

    if (!full && gbs_generic_smem_bytes(p, nullptr) > (size_t)p->smem_optin) { delete p; return GBS_ERR_UNSUPPORTED; }

    e = cudaMalloc(&p->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, sizeof(int));
    if (e != cudaSuccess) { cudaGetLastError(); if (p->d_status) cudaFree(p->d_status); delete p; return GBS_ERR_ALLOC; }
    if (full) {
        // the only family for a full order: the bf16 image of H_m (m * m * 2 bytes) is the plan's one table
        if (!gbs_tc_dense_supported(p)) { cudaFree(p->d_status); delete p; return GBS_ERR_UNSUPPORTED; }
        int8_t* hm = (int8_t*)malloc((size_t)m * m);
        unsigned short* img = (unsigned short*)malloc((size_t)m * m * 2);
        rc = (hm && img) ? gbs_build_hadamard_m(m, hm) : GBS_ERR_ALLOC;
        if (rc == GBS_OK) {
            gbs_tc_dense_image(hm, m, img);
            e = cudaMalloc(&p->d_aimg, (size_t)m * m * 2);
            if (e == cudaSuccess) e = cudaMemcpy(p->d_aimg, img, (size_t)m * m * 2, cudaMemcpyHostToDevice);
            if (e != cudaSuccess) { cudaGetLastError(); rc = GBS_ERR_ALLOC; }
        }
        free(hm);
        free(img);
        if (rc != GBS_OK) {
            if (p->d_aimg) cudaFree(p->d_aimg);
            cudaFree(p->d_status);
            delete p;
            return rc;
        }
        p->variant = GBS_VARIANT_TC_DENSE;
        p->pdl = 0;
        *out = p;
        return GBS_OK;
    }
    const char* force = getenv("GBS_FORCE_GENERIC");
    const bool want_tc = !(force && force[0] == '1');
    const bool tc_uv = want_tc && gbs_tc_uv_supported(p);
    const bool tc_row = want_tc && !tc_uv && gbs_tc_row_supported(p);
    const int uvm_glog = (want_tc && !tc_uv && !tc_row) ? gbs_tc_uvm_glog(p) : 0;
    if (tc_uv || tc_row || uvm_glog) {
        // the UV family with one symmetric scale per token also gets the image of the transpose, behind the
        // first one in the same allocation, for gbs_dequantize's inverse rotation on the tensor cores
        const bool with_t = tc_uv && p->group == 0 && !p->asym;
        // the wide family keeps the UVM image (clip scoring) and, where the register-resident kernel applies, its image
        const char* no_uvr = getenv("GBS_NO_UVR");
        const bool uvr = uvm_glog != 0 && !(no_uvr && no_uvr[0] == '1') && gbs_tc_uvr_supported(p);
        const size_t img_bytes = with_t ? 65536 : (uvr ? 32768 + (size_t)gbs_tc_uvr_image_bytes(p) : 32768);
        unsigned char* img = (unsigned char*)malloc(img_bytes);
        if (!img) { cudaFree(p->d_status); delete p; return GBS_ERR_ALLOC; }
        if (tc_uv) gbs_tc_uv_a_image(p, img);
        if (with_t) {
            const int j = p->k - 5, U = p->d_pad / 32;
            gbs_tc_sign_image(p->h_hm, p->m, j, U, img + 32768, true);
            for (int c = 0; c < U; ++c) {
                int sum = 0;
                for (int r = 0; r < U; ++r) {
                    int sign = p->h_hm[(r >> j) * p->m + (c >> j)];
                    if (__builtin_popcount((unsigned)(r & c & ((1 << j) - 1))) & 1) sign = -sign;
                    sum += sign;
                }
                p->a_colsum[c] = sum;
            }
        }
        else if (tc_row) gbs_tc_sign_image(p->h_hm, 1, 7, 128, img);     // H_128 itself
        else gbs_tc_sign_image(p->h_hm, p->m, p->k - 5 - uvm_glog, p->d_pad >> (5 + uvm_glog), img);
        if (uvr) gbs_tc_uvr_image(p, img + 32768);
        e = cudaMalloc(&p->d_aimg, img_bytes);
        if (e == cudaSuccess) e = cudaMemcpy(p->d_aimg, img, img_bytes, cudaMemcpyHostToDevice);
        free(img);
        if (e == cudaSuccess && with_t) p->d_aimg_t = p->d_aimg + 32768;
        if (e == cudaSuccess && uvr) p->d_aimg_r = p->d_aimg + 32768;
        if (e != cudaSuccess) {
            cudaGetLastError();
            if (p->d_aimg) cudaFree(p->d_aimg);
            cudaFree(p->d_status); delete p; return GBS_ERR_ALLOC;
        }
        p->variant = tc_uv ? GBS_VARIANT_TC_UV : (tc_row ? GBS_VARIANT_TC_ROW : (uvr ? GBS_VARIANT_TC_UVR : GBS_VARIANT_TC_UVM));
        p->uvm_glog = uvm_glog;
    }
    if (p->asym && p->variant != GBS_VARIANT_TC_ROW) {          // only the row family has the asymmetric quantizer
        if (p->d_aimg) cudaFree(p->d_aimg);
        cudaFree(p->d_status);
        delete p;
        return GBS_ERR_UNSUPPORTED;
    }
    const char* nopdl = getenv("GBS_NO_PDL");
    p->pdl = (nopdl && nopdl[0] == '1') ? 0 : 1;

    if (m > 1) {
        float* h = new (std::nothrow) float[(size_t)2 * m * m];
        if (!h) { cudaFree(p->d_status); if (p->d_aimg) cudaFree(p->d_aimg); delete p; return GBS_ERR_ALLOC; }
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) {
                h[i * m + j] = (float)p->h_hm[i * m + j];
                h[m * m + j * m + i] = (float)p->h_hm[i * m + j];     // transpose, for the inverse rotation
            }
        e = cudaMalloc(&p->d_hm, sizeof(float) * 2 * m * m);
        if (e != cudaSuccess) { delete[] h; cudaGetLastError(); cudaFree(p->d_status); if (p->d_aimg) cudaFree(p->d_aimg); delete p; return GBS_ERR_ALLOC; }
        e = cudaMemcpy(p->d_hm, h, sizeof(float) * 2 * m * m, cudaMemcpyHostToDevice);
        delete[] h;
        if (e != cudaSuccess) { cudaGetLastError(); cudaFree(p->d_hm); cudaFree(p->d_status); if (p->d_aimg) cudaFree(p->d_aimg); delete p; return GBS_ERR_CUDA; }
    }
    *out = p;
    return GBS_OK;
}

extern "C" int gbs_plan_destroy(gbs_plan_t* plan)
{
    if (!plan) return GBS_OK;
    int rc = GBS_OK;
    {
        DeviceGuard g;
        if (g.enter(plan->device) != cudaSuccess) { cudaGetLastError(); rc = GBS_ERR_CUDA; }
        else {
            if (plan->d_hm && cudaFree(plan->d_hm) != cudaSuccess) { cudaGetLastError(); rc = GBS_ERR_CUDA; }
            if (plan->d_status && cudaFree(plan->d_status) != cudaSuccess) { cudaGetLastError(); rc = GBS_ERR_CUDA; }
            if (plan->d_aimg && cudaFree(plan->d_aimg) != cudaSuccess) { cudaGetLastError(); rc = GBS_ERR_CUDA; }
        }
    }
    delete plan;
    return rc;
}

extern "C" int gbs_plan_info(const gbs_plan_t* p, gbs_plan_info_t* out)
{
    if (!p || !out) return GBS_ERR_INVALID_ARG;
    out->d = p->d; out->d_pad = p->d_pad; out->m = p->m; out->k = p->k;
    out->bits = p->bits; out->group = p->group; out->alpha = p->alpha;
    out->levels = p->levels; out->q_lo = -p->levels; out->q_hi = p->levels;
    out->code_bytes_per_row = (int64_t)p->d_pad * p->bits / 8;
    out->scales_per_row = p->group ? p->d_pad / p->group : 1;
    out->asymmetric = p->asym;
    out->scale_floats_per_row = out->scales_per_row * (p->asym ? 2 : 1);
    out->variant = p->variant;
    return GBS_OK;
}

extern "C" int gbs_plan_device_status(const gbs_plan_t* p, int* out)
{
    if (!p || !out) return GBS_ERR_INVALID_ARG;
    DeviceGuard g;
    if (g.enter(p->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    int v = 0;
    if (cudaMemcpy(&v, p->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(p->d_status, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return GBS_ERR_CUDA;
    }
    *out = v;
    return GBS_OK;
}

extern "C" int gbs_rotate_quantize(const gbs_plan_t* p, const void* x, int x_dtype, int64_t n_rows,
                                   int64_t x_row_stride, void* codes, float* scales, float* y_opt,
                                   void* cuda_stream)
{
    int rc = check_rows(p, x, x_dtype, n_rows, x_row_stride);
    if (rc != GBS_OK || n_rows == 0) return rc;
    if (!codes || !scales) return GBS_ERR_INVALID_ARG;
    if (!aligned16(codes) || (y_opt && !aligned16(y_opt)) || (reinterpret_cast<uintptr_t>(scales) & 3u))
        return GBS_ERR_ALIGNMENT;
    if (p->asym && !(p->variant == GBS_VARIANT_TC_ROW && x_dtype == GBS_DTYPE_BF16)) return GBS_ERR_UNSUPPORTED;
    if (p->variant == GBS_VARIANT_TC_DENSE && x_dtype != GBS_DTYPE_BF16) return GBS_ERR_UNSUPPORTED;   // bf16 rows only
    DeviceGuard g;
    if (g.enter(p->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int e;
    if (p->variant == GBS_VARIANT_TC_DENSE)
        e = gbs_tc_dense_rotate_quantize(p, x, n_rows, x_row_stride, codes, scales, y_opt, stream);
    else if (p->variant == GBS_VARIANT_TC_UV && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_uv_rotate_quantize(p, x, n_rows, x_row_stride, codes, scales, y_opt, stream);
    else if (p->variant == GBS_VARIANT_TC_UVR && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_uvr_rotate_quantize(p, x, n_rows, x_row_stride, codes, scales, y_opt, stream);
    else if (p->variant == GBS_VARIANT_TC_UVM && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_uvm_rotate_quantize(p, x, n_rows, x_row_stride, codes, scales, y_opt, stream);
    else if (p->variant == GBS_VARIANT_TC_ROW && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_row_rotate_quantize(p, x, n_rows, x_row_stride, codes, scales, y_opt, stream);
    else
        e = gbs_generic_rotate_quantize(p, x, x_dtype, n_rows, x_row_stride, codes, scales, y_opt, stream);
    if (e != 0) cudaGetLastError();
    return e == 0 ? GBS_OK : GBS_ERR_CUDA;
}

extern "C" int gbs_dequantize(const gbs_plan_t* p, const void* codes, const float* scales, int64_t n_rows,
                              void* out, int out_dtype, int flags, void* cuda_stream)
{
    if (!p) return GBS_ERR_INVALID_ARG;
    if (out_dtype != GBS_DTYPE_F32 && out_dtype != GBS_DTYPE_BF16) return GBS_ERR_INVALID_ARG;
    if (flags & ~GBS_INVERSE_ROTATE) return GBS_ERR_INVALID_ARG;
    if (n_rows < 0) return GBS_ERR_INVALID_ARG;
    if ((flags & GBS_INVERSE_ROTATE) && p->variant == GBS_VARIANT_TC_DENSE && !gbs_tc_denseinv_supported(p)) return GBS_ERR_UNSUPPORTED;
    if (n_rows == 0) return GBS_OK;
    if (!codes || !scales || !out) return GBS_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(out) || (reinterpret_cast<uintptr_t>(scales) & 3u))
        return GBS_ERR_ALIGNMENT;
    DeviceGuard g;
    if (g.enter(p->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    int e;
    if ((flags & GBS_INVERSE_ROTATE) && p->variant == GBS_VARIANT_TC_DENSE)
        e = gbs_tc_denseinv_dequantize(p, codes, scales, n_rows, out, out_dtype, static_cast<cudaStream_t>(cuda_stream));
    else if ((flags & GBS_INVERSE_ROTATE) && gbs_tc_uvinv_supported(p))
        e = gbs_tc_uvinv_dequantize(p, codes, scales, n_rows, out, out_dtype, static_cast<cudaStream_t>(cuda_stream));
    else if ((flags & GBS_INVERSE_ROTATE) && gbs_tc_rowinv_supported(p, scales))
        e = gbs_tc_rowinv_dequantize(p, codes, scales, n_rows, out, out_dtype, static_cast<cudaStream_t>(cuda_stream));
    else
        e = gbs_generic_dequantize(p, codes, scales, n_rows, out, out_dtype, (flags & GBS_INVERSE_ROTATE) != 0,
                                   static_cast<cudaStream_t>(cuda_stream));
    return e == 0 ? GBS_OK : GBS_ERR_CUDA;
}

extern "C" int gbs_clip_error(const gbs_plan_t* p, const void* x, int x_dtype, int64_t n_rows,
                              int64_t x_row_stride, const float* alphas_host, int K, double* err_sum,
                              float* err_rows_opt, void* cuda_stream)
{
    int rc = check_rows(p, x, x_dtype, n_rows, x_row_stride);
    if (rc != GBS_OK) return rc;
    if (K < 1 || K > GBS_MAX_CANDIDATES || !alphas_host) return GBS_ERR_INVALID_ARG;
    if (p->asym || p->variant == GBS_VARIANT_TC_DENSE) return GBS_ERR_UNSUPPORTED;
    float c_scale[GBS_MAX_CANDIDATES], c_inv[GBS_MAX_CANDIDATES];
    const double rootn = sqrt((double)p->d_pad);
    for (int i = 0; i < K; ++i) {
        const float a = alphas_host[i];
        if (!(a > 0.f) || !(a <= 1.f)) return GBS_ERR_INVALID_ARG;
        c_scale[i] = (float)((double)a / ((double)p->levels * rootn));
        c_inv[i] = (float)((double)p->levels / (double)a);
    }
    if (n_rows == 0) return GBS_OK;
    if (!err_sum) return GBS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(err_sum) & 7u) || (err_rows_opt && (reinterpret_cast<uintptr_t>(err_rows_opt) & 3u)))
        return GBS_ERR_ALIGNMENT;
    DeviceGuard g;
    if (g.enter(p->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    int e;
    if (p->variant == GBS_VARIANT_TC_UV && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_uv_clip_error(p, x, n_rows, x_row_stride, alphas_host, K, err_sum, err_rows_opt,
                                 static_cast<cudaStream_t>(cuda_stream));
    else if (p->variant == GBS_VARIANT_TC_ROW && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_row_clip_error(p, x, n_rows, x_row_stride, alphas_host, K, err_sum, err_rows_opt,
                                  static_cast<cudaStream_t>(cuda_stream));
    else if ((p->variant == GBS_VARIANT_TC_UVM || p->variant == GBS_VARIANT_TC_UVR) && x_dtype == GBS_DTYPE_BF16)
        e = gbs_tc_uvm_clip_error(p, x, n_rows, x_row_stride, alphas_host, K, err_sum, err_rows_opt,
                                  static_cast<cudaStream_t>(cuda_stream));
    else
        e = gbs_generic_clip_error(p, x, x_dtype, n_rows, x_row_stride, c_scale, c_inv, K, err_sum, err_rows_opt,
                                   static_cast<cudaStream_t>(cuda_stream));
    if (e != 0) cudaGetLastError();
    return e == 0 ? GBS_OK : GBS_ERR_CUDA;
}
