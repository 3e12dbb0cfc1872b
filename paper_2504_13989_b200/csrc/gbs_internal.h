// Internal declarations shared by the translation units of libgbs (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "gbs.h"

// Largest order of the small Hadamard factor H_m a plan accepts.
#define GBS_MAX_M 108

// Kernel families a plan can select for bf16 rows.
enum gbs_variant {
    GBS_VARIANT_GENERIC = 0,   // shared-memory FWHT on the plain ALUs; any supported (m, k), any dtype
    GBS_VARIANT_TC_UVM = 3,    // 4096 < d' = 32*G*U <= 32768, G in {2,4,8}: tensor cores + two register sweeps over TMEM
    GBS_VARIANT_TC_ROW = 2,    // d' = 128 (KV rows): X * H_128 on tcgen05 tensor cores, one thread owns one row
    GBS_VARIANT_TC_UVR = 5,    // 4096 < d' = 128*U <= 32768, 80 <= U <= 256: tensor cores + the rest of the transform in registers
    GBS_VARIANT_TC_DENSE = 4,  // d' = m, a full Paley order (k = 0): X * H_m^T as a dense tcgen05 contraction, two sweeps
    GBS_VARIANT_TC_UV = 1,     // d' = U*32, U = m*2^j <= 128: (H_m (x) H_{2^j}) on tcgen05 tensor cores + H_32 in
                               // registers (bf16 rows)
};

struct gbs_plan {
    int d, d_pad, m, k;
    int bits, group;
    float alpha;
    int levels;            // D
    float norm;            // 1/sqrt(d')
    float c_scale;         // alpha / (D sqrt(d')):  Delta = c_scale * max|Y|   (Y = unnormalised rotation)
    float c_inv;           // D / alpha:             code  = rint(Y * c_inv / max|Y|)
    int device;
    int sm_count;
    int smem_optin;        // largest dynamic shared memory a block may opt in to
    int variant;
    float* d_hm;           // device: H_m as floats, m*m row-major, followed by H_m^T (m*m)
    int pdl;               // tensor-core families launch with programmatic stream serialization
    int asym;              // asymmetric quantizer (GBS_PLAN_ASYMMETRIC)
    int uvm_glog;          // UVM family: log2 of the number of 32-value chunks per tensor-core output row
    unsigned char* d_aimg; // device: pre-swizzled bf16 image of H_m (x) H_{2^j} for the tensor-core family (32 KB)
    unsigned char* d_aimg_r; // device: image of H_m (x) H_{2^j} for the UVR family (behind the first one), or null
    unsigned char* d_aimg_t; // device: image of its transpose (UV family, one scale per token: inverse rotation), or null
    int a_colsum[128];     // column sums of H_m (x) H_{2^j} (UV family), for the inverse path's offset correction
    int* d_status;         // device status word: 0, or the code of the first bounded wait that expired
    int8_t h_hm[GBS_MAX_M * GBS_MAX_M];  // host copy of H_m
};

// Makes `dev` the current device for the lifetime of the object (entry points work on the plan's device).
struct gbs_device_guard {
    int prev = -1;
    bool switched = false;
    cudaError_t enter(int dev)
    {
        cudaError_t e = cudaGetDevice(&prev);
        if (e != cudaSuccess) return e;
        if (prev != dev) {
            e = cudaSetDevice(dev);
            switched = (e == cudaSuccess);
        }
        return e;
    }
    ~gbs_device_guard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

// gbs_paley.cu
int gbs_build_hadamard_m(int m, int8_t* out);   // 0 or GBS_ERR_UNSUPPORTED
bool gbs_supported_m(int m);                    // the orders a plan accepts as the factor of H_m (x) H_{2^k}
bool gbs_supported_full_m(int m);               // the orders a plan accepts as the whole rotation (d' = m, k = 0)

// gbs_generic.cu : launches on `stream`; return a cudaError_t cast to int (0 = success)
int gbs_generic_rotate_quantize(const gbs_plan* p, const void* x, int x_dtype, int64_t n_rows,
                                int64_t stride, void* codes, float* scales, float* y_opt,
                                cudaStream_t stream);
int gbs_generic_clip_error(const gbs_plan* p, const void* x, int x_dtype, int64_t n_rows,
                           int64_t stride, const float* c_scale_k, const float* c_inv_k, int K,
                           double* err_sum, float* err_rows, cudaStream_t stream);
int gbs_generic_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows,
                           void* out, int out_dtype, int inverse, cudaStream_t stream);
size_t gbs_generic_smem_bytes(const gbs_plan* p, int* rows_per_cta);

// gbs_tc_uvinv.cu : gbs_dequantize with inverse rotation on the tensor cores
bool gbs_tc_uvinv_supported(const gbs_plan* p);
int gbs_tc_uvinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                            int out_dtype, cudaStream_t stream);

// gbs_tc_rowinv.cu : the same for d' = 128 rows with one scale (pair) per row
bool gbs_tc_rowinv_supported(const gbs_plan* p, const float* scales);
int gbs_tc_rowinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                             int out_dtype, cudaStream_t stream);

// gbs_tc_uv.cu
bool gbs_tc_uv_supported(const gbs_plan* p);
int gbs_tc_uv_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                         double* err_sum, float* err_rows, cudaStream_t stream);
void gbs_tc_uv_a_image(const gbs_plan* p, unsigned char* img32k);
// image of H_m (x) H_{2^j} (U x U inside 128 x 128, bf16 +-1, K-major, 128-byte swizzle)
void gbs_tc_sign_image(const int8_t* hm, int m, int j, int U, unsigned char* img32k, bool transpose = false);

int gbs_tc_row_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                          double* err_sum, float* err_rows, cudaStream_t stream);

// gbs_tc_uvm.cu
int gbs_tc_uvm_glog(const gbs_plan* p);        // 0 if the family does not apply
int gbs_tc_uvm_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream);
int gbs_tc_uvm_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                          double* err_sum, float* err_rows, cudaStream_t stream);

// gbs_tc_uvr.cu : rotate-quantize for wide rows with the register-resident epilogue (clip scoring stays with UVM)
bool gbs_tc_uvr_supported(const gbs_plan* p);
int gbs_tc_uvr_image_bytes(const gbs_plan* p);
void gbs_tc_uvr_image(const gbs_plan* p, unsigned char* img);
int gbs_tc_uvr_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream);

// gbs_tc_dense.cu
bool gbs_tc_dense_supported(const gbs_plan* p);
void gbs_tc_dense_image(const int8_t* hm, int m, unsigned short* img);
int gbs_tc_dense_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                                 float* scales, float* y_opt, cudaStream_t stream);

// gbs_tc_denseinv.cu : gbs_dequantize with inverse rotation for the full order
bool gbs_tc_denseinv_supported(const gbs_plan* p);
int gbs_tc_denseinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                               int out_dtype, cudaStream_t stream);

// gbs_tc_row.cu
bool gbs_tc_row_supported(const gbs_plan* p);
int gbs_tc_row_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream);
int gbs_tc_uv_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                              float* scales, float* y_opt, cudaStream_t stream);
