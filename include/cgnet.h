/* cgnet -- the ungated glue of a channel-gated ResNet: the operations between the gated
 * convolution layers of cgconv.h when a whole network runs on the device.
 *
 * "Channel Gating Neural Networks" (arXiv 1805.12549) gates the convolution layers of standard
 * networks (Section 5: ResNet-18 and others) and leaves the remaining operators as they are:
 * the stem convolution, the pooling layers and the classifier.  These entry points are those
 * operators for a ResNet-18 in NHWC bf16; every one is a single memory-bound kernel.
 *
 * All pointers are DEVICE pointers owned by the caller, 16-byte aligned; nothing is allocated;
 * each call enqueues one kernel on `cuda_stream` and returns without synchronising.  Return
 * values are cg_status codes (cgconv.h): CG_ERR_INVALID_ARG for NULL pointers or non-positive
 * extents, CG_ERR_ALIGNMENT, CG_ERR_CUDA for a failed launch.
 */
#ifndef CGNET_H_
#define CGNET_H_

#include "cgconv.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Patch matrix of a convolution (the stem: 7x7, stride 2, 3 channels).
 * x [n,h,w,c] bf16  ->  a [n,h',w',k_pad] bf16 with h' = (h + 2*pad - k)/stride + 1 (w' alike),
 * a[n,i,j,(r*k + s)*c + ci] = x[n, i*stride + r - pad, j*stride + s - pad, ci], zero outside the
 * image, zero for the columns k*k*c .. k_pad-1.  k_pad >= k*k*c and a multiple of 8.
 * A 1x1 gated layer (groups = 1) over `a` with the filter reshaped to [c_out, k_pad] is then the
 * convolution itself, with its batch norm and ReLU fused. */
cg_status cg_im2col_bf16(const void* x, void* a, int n, int h, int w, int c, int k, int stride,
                         int pad, int k_pad, void* cuda_stream);

/* Every stride-th pixel: y[n,i,j,:] = x[n,i*stride,j*stride,:], y is [n,ceil(h/stride),
 * ceil(w/stride),c].  Input of the 1x1 stride-2 shortcut convolutions.  c a multiple of 8. */
cg_status cg_subsample_bf16(const void* x, void* y, int n, int h, int w, int c, int stride,
                            void* cuda_stream);

/* Max pooling k x k, given stride and padding (padding never wins: it counts as -inf).
 * y is [n,(h + 2*pad - k)/stride + 1,(w + 2*pad - k)/stride + 1,c].  c a multiple of 8. */
cg_status cg_maxpool_bf16(const void* x, void* y, int n, int h, int w, int c, int k, int stride,
                          int pad, void* cuda_stream);

/* Global average pooling: y[n,c] = mean over the h*w pixels of x[n,:,:,c], summed in fp32 in
 * pixel order and rounded to bf16 once.  c a multiple of 8. */
cg_status cg_avgpool_bf16(const void* x, void* y, int n, int hw, int c, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CGNET_H_ */
