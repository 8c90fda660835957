/*
 * dft3d -- 3D complex-to-complex discrete Fourier transform on one NVIDIA B200,
 * computed as dense matrix multiplications on the tensor cores.
 *
 * Two formulations of the same transform (both from "Large-Scale Discrete
 * Fourier Transform on TPUs", arXiv 2002.03260):
 *
 *   KDFT (Section III-A, Eq. 11-13): every axis is multiplied by its N x N
 *        Vandermonde / DFT matrix.  The matrix may be built from nonuniform
 *        sample nodes (Eq. 3 with the sample points on the unit circle).
 *   FFT  (Section III-B, Eq. 14-18): every axis of length N = N1*N2 becomes a
 *        length-N1 DFT (matrix product), an elementwise phase adjustment
 *        (twiddle), and a length-N2 DFT (matrix product); output in natural
 *        order.  Uniform grids only.  (Lengths above 1024 apply Eq. 17 once
 *        more, with a factor 2, 4 or 8 whose small DFT runs on the CUDA cores.)
 *
 * Data layout everywhere: row-major [n0][n1][n2], interleaved complex64
 * (re, im as two float32), 8 bytes per point.
 *
 * All functions return a DFT3D_* status and never throw or abort.  A short
 * description of the most recent failure on the calling thread is available
 * from dft3d_last_error().
 */
#ifndef DFT3D_H_
#define DFT3D_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dft3d_plan_s* dft3d_plan_t;

enum { DFT3D_KDFT = 0, DFT3D_FFT = 1, DFT3D_AUTO = 2 }; /* mode; AUTO: per axis, FFT where it applies, else KDFT */
enum { DFT3D_FORWARD = -1, DFT3D_INVERSE = +1 }; /* sign of the exponent (Eq. 14 has the minus sign) */

enum {
  DFT3D_OK = 0,
  DFT3D_ERR_INVALID_ARG = 1,    /* NULL where not allowed, n < 1, bad mode/sign, non-finite node, misaligned pointer */
  DFT3D_ERR_UNSUPPORTED = 2,    /* size or option outside what the kernels handle (see dft3d_plan_create) */
  DFT3D_ERR_ALLOC = 3,          /* host or device allocation failed */
  DFT3D_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed */
  DFT3D_ERR_DEVICE_TIMEOUT = 5  /* a kernel gave up a bounded wait; the output of that execute is invalid */
};

/* option flags */
enum {
  DFT3D_NODES_ON_OUTPUT = 1u,   /* M[k,j] = exp(s*2*pi*i * node[k] * j): Eq. 1 read literally (arbitrary
                                   evaluation points, integer powers).  Default is M[k,j] = exp(s*2*pi*i * k * node[j])
                                   (nonuniform input samples, integer output frequencies). */
  DFT3D_UNSCALED_INVERSE = 2u,  /* sign=+1 without the 1/n_a factors */
  /* Operand split of the tensor-core products (Section II-A: float32 accuracy from several reduced-precision
     pieces whose products are accumulated).  Both use 3
     products of 11-bit pieces with fp32 accumulation and meet the same error bound.  Default: fp16 pieces (KDFT:
     when every transformed n_a % 4 == 0, TF32 pieces otherwise). */
  DFT3D_SPLIT_FP16 = 4u,        /* insist on fp16 pieces (operands scaled by exact powers of two: KDFT from the largest
                                   input magnitude, FFT per line; half the tensor-core instructions of TF32);
                                   DFT3D_ERR_UNSUPPORTED for KDFT when a transformed n_a is not a multiple of 4 */
  DFT3D_SPLIT_TF32 = 8u,        /* insist on TF32 pieces (no scaling; every element keeps ~22 significant bits
                                   whatever the dynamic range of the input) */
  DFT3D_DESTROY_INPUT = 16u,    /* dft3d_execute may overwrite `in`: a plan over all three axes then uses the input
                                   cube as its workspace and allocates none, which keeps the fast schedules available
                                   when input + output fill the memory (2048^3).  Ignored by plans over fewer axes. */
  DFT3D_INVERSE_SOLVE = 32u     /* KDFT, sign = +1, axes with nodes: the true inverse of the nonuniform transform
                                   (Section III-A: for points that are not roots of unity the inverse is the
                                   solution of the linear system of Eq. 2).  The n_a x n_a forward matrix of the nodes is inverted
                                   once at plan creation (float64, on the host; n_a <= 2048) and the solve becomes
                                   one more matrix product, so inverse(forward(x)) = x for distinct nodes.  Axes
                                   without nodes use the usual scaled inverse, which is that inverse.  Singular or
                                   hopelessly ill-conditioned node sets are refused. */
};

typedef struct dft3d_options_s {
  size_t struct_size;     /* sizeof(dft3d_options_t), for forward compatibility */
  unsigned flags;         /* DFT3D_NODES_ON_OUTPUT | DFT3D_UNSCALED_INVERSE | DFT3D_SPLIT_* | DFT3D_DESTROY_INPUT */
  int fft_split[3][2];    /* FFT mode: {N1, N2} per axis with N1*N2 = n_a, first and second matrix product of Eq. 17.
                             {0,0} = the built-in split, which is also the only one the kernels realise: N2 = 16 for
                             n_a = 256 and 512, N2 = 32 from 1024 on, N1 = n_a / N2 (256 = 16*16, 512 = 32*16,
                             1024 = 32*32, 2048 = 64*32, 4096 = 128*32; an N1 above N2 is itself computed as
                             (N1/N2) * N2 by one more application of Eq. 17; 8192 = 1024*8, the 1024 again 32*32).
                             Any other pair returns
                             DFT3D_ERR_UNSUPPORTED; dft3d_plan_fft_split reports the pair in use. */
  size_t workspace_limit; /* upper bound in bytes for the plan-owned workspace; 0 = default (16 GiB).  KDFT needs a
                             workspace and shrinks it to groups of n0-planes.  FFT uses one cube of workspace when it
                             fits (fewest launches), else a half, a quarter or an eighth of a cube, whichever fits
                             first (fp16 pieces: the strided passes run once per slice of the last axis), and
                             otherwise runs in place on `out`. */
  unsigned axes;          /* bit a set = transform axis a; 0 = all three.  6 (axes 1 and 2) is a batch of n0
                             two-dimensional transforms (Eq. 5), 4 a batch of n0*n1 one-dimensional ones (Eq. 2).
                             An axis that is not transformed may have any length >= 1 if it is axis 0. */
} dft3d_options_t;

/*
 * Create a plan for an n0 x n1 x n2 transform (Eq. 11 / Eq. 12).
 *
 *   out      receives the handle; set to NULL on failure.
 *   mode     DFT3D_KDFT, DFT3D_FFT, or DFT3D_AUTO: the FFT formulation on every transformed axis that has a uniform
 *            grid, a length the FFT kernels take and at least 16 neighbouring lines, the KDFT formulation on the
 *            others (nonuniform nodes, other even lengths).  A plan that ends up with both needs one cube of
 *            workspace (or DFT3D_DESTROY_INPUT) and runs every pass in the natural layout.
 *   sign     DFT3D_FORWARD: kernel exp(-2*pi*i*k*t), unscaled (Eq. 14).
 *            DFT3D_INVERSE: conjugate kernel, each axis scaled by 1/n_a so that
 *            inverse(forward(x)) = x on uniform grids (the paper describes the inverse
 *            as solving Eq. 2; on a uniform grid that solve is this product).
 *   nodesA   HOST pointer to n_a doubles, or NULL for the uniform grid t_j = j/n_a.
 *            Any finite value is accepted and used modulo 1.  Copied during the call.
 *            With nodes and sign=+1 the result is the conjugate-kernel product (see DFT3D_INVERSE_SOLVE), not an
 *            inverse of the nonuniform transform.  FFT mode takes no nodes.
 *
 * The DFT / Vandermonde matrices and twiddles are evaluated in float64 with exactly
 * reduced phases and rounded once to the stored float32 pieces.  The plan owns its
 * device tables and workspace (allocated on the current device during this call).
 *
 * Supported sizes: KDFT: n0 and n1 of any length, n2 even (rows of the data must start on 16-byte boundaries),
 * transformed n_a <= 8192 (tiles that are not full are zero-filled on load and masked on store, and an odd length pads
 * the rows of the table, the way the paper's compiler pads to its hardware's preferred shapes).  FFT: every
 * transformed n_a in {256, 512, 1024, 2048, 4096, 8192} (N = R*R, 2*R*R or 4*R*R with R = 16 or 32, and 8192 = 1024*8;
 * 4096 and 8192 with fp16 pieces only), the others multiples of 64.  An 8192-point axis takes two launches (the fused
 * 1024-point kernel over the eight stride-8 sub-sequences, then the phase adjustment and the 8-point DFT), and a plan
 * that has one owns a cube of workspace and runs its axes one after the other in the natural layout.
 * Other sizes return DFT3D_ERR_UNSUPPORTED.
 */
int dft3d_plan_create(dft3d_plan_t* out, long long n0, long long n1, long long n2, int mode, int sign,
                      const double* nodes0, const double* nodes1, const double* nodes2);

/* Same, with options (may be NULL). */
int dft3d_plan_create_ex(dft3d_plan_t* out, long long n0, long long n1, long long n2, int mode, int sign,
                         const double* nodes0, const double* nodes1, const double* nodes2,
                         const dft3d_options_t* options);

/*
 * Run the transform (all three axes; Eq. 12 for KDFT, Eq. 17 per axis for FFT).
 *
 *   in, out      DEVICE pointers, 16-byte aligned, n0*n1*n2*8 bytes each, not overlapping.
 *                `in` is only read, unless the plan was created with DFT3D_DESTROY_INPUT.
 *   cuda_stream  a cudaStream_t (NULL = default stream).
 *
 * Asynchronous: kernels are enqueued on the stream and the call returns without
 * synchronising.  No allocation happens here, and nothing is read back from the device, so the
 * call may be captured into a CUDA graph and replayed on new data in the same buffers.
 * One execute per plan may be in flight.
 * After the stream has been synchronised, dft3d_plan_status() tells whether any kernel
 * abandoned a bounded wait.
 */
int dft3d_execute(dft3d_plan_t plan, const void* in, void* out, void* cuda_stream);

/*
 * Convenience for callers whose data lives in HOST memory (pinned memory makes the copies
 * faster): copies `host_in` to a plan-owned device buffer, runs dft3d_execute, copies the
 * result to `host_out`, and synchronises the stream before returning.  The device buffers
 * are allocated on first use and kept until the plan is destroyed.
 */
int dft3d_execute_host(dft3d_plan_t plan, const void* host_in, void* host_out, void* cuda_stream);

/*
 * A sequence of `count` transforms of HOST cubes, streamed: host_in[i] / host_out[i] are HOST pointers to cubes of
 * the plan's shape (pinned memory, or the copies cannot overlap anything).  Two plan-owned pairs of device buffers
 * take turns, the uploads and the downloads run on two plan-owned streams, the transforms on `cuda_stream`: the
 * download of cube i and the upload of cube i+1 use the two directions of the link at the same time, under the
 * transform of whichever cube is on the device.  Results are the same as `count` calls of dft3d_execute_host (same
 * kernels, same order per cube).  The same host buffer may appear several times in host_out (later results
 * overwrite earlier ones, in order); a host_in buffer must not be one of the host_out buffers.  Synchronous:
 * returns after the last download; status as dft3d_execute_host.  The extra device buffers and the streams are
 * created on first use and kept until the plan is destroyed.  count == 0 is a no-op.
 */
int dft3d_execute_host_batch(dft3d_plan_t plan, const void* const* host_in, void* const* host_out, int count,
                             void* cuda_stream);

/* Transform one axis only (0, 1 or 2) with the plan's matrix for that axis; same pointer rules as
 * dft3d_execute.  KDFT: Eq. 5's left / right multiplication for that axis.  FFT: Eq. 17 along that axis. */
int dft3d_execute_axis(dft3d_plan_t plan, int axis, const void* in, void* out, void* cuda_stream);

/* DFT3D_OK, or DFT3D_ERR_DEVICE_TIMEOUT if a kernel of an earlier execute gave up a wait.
 * Reads a plan-owned device word (a small synchronous copy); call it after synchronising. */
int dft3d_plan_status(dft3d_plan_t plan);

/* Bytes of device workspace the plan owns (0 for NULL). */
size_t dft3d_plan_workspace_bytes(dft3d_plan_t plan);

/* Number of kernels one dft3d_execute enqueues (0 for NULL).  KDFT with fp16 pieces: this counts the small
 * reduction that finds the largest input magnitude before the first axis pass.  FFT: 3 for a 3D transform, or
 * 2 * slices + 1 when the workspace holds only a half, a quarter or an eighth of a cube. */
int dft3d_plan_launches(dft3d_plan_t plan);

/* DFT3D_SPLIT_FP16 or DFT3D_SPLIT_TF32: the operand split the plan uses; 0 for NULL. */
int dft3d_plan_split(dft3d_plan_t plan);

/* The factor pair {N1, N2} of Eq. 17 that the plan uses on `axis` (N1 * N2 = n_axis): DFT3D_OK and the pair for an axis
 * the plan transforms in the FFT formulation, DFT3D_ERR_INVALID_ARG otherwise (NULL plan or pointers, an axis in the KDFT
 * formulation or not transformed). */
int dft3d_plan_fft_split(dft3d_plan_t plan, int axis, int* n1, int* n2);

/* Frees device and host memory of the plan.  NULL is accepted. */
int dft3d_plan_destroy(dft3d_plan_t plan);

const char* dft3d_status_string(int status);
const char* dft3d_last_error(void);

/*
 * The table generator, exposed so that it can be checked on a machine without a GPU
 * (HOST pointers only; no CUDA call is made).
 *
 * dft3d_generate_axis_matrix: the n x n complex matrix of one axis in float64,
 *   M[k][j] interleaved (re, im), 2*n*n doubles.  (Eq. 3 / Eq. 13; Eq. 14 when nodes == NULL.)
 * dft3d_generate_twiddle: T[k1][beta] = exp(sign*2*pi*i*k1*beta/(N1*N2)), N1*N2 complex doubles
 *   (the phase adjustment of Eq. 17).
 * dft3d_generate_real_table: the real 2n x 2n matrix W with W[2k+p][2j+q] =
 *   (p==q ? Re M[k][j] : (p ? +Im : -Im) M[k][j]) that turns the complex product into a real
 *   one on interleaved data, split into two float32 pieces hi + lo (hi has a 10-bit
 *   mantissa, i.e. is exact in TF32; lo is the float32 rounding of the remainder rounded to
 *   TF32).  Each piece is (2n)*(2n) floats, row-major.
 */
int dft3d_generate_axis_matrix(long long n, int sign, double scale, const double* nodes, int nodes_on_output,
                               double* matrix);
int dft3d_generate_twiddle(long long N1, long long N2, int sign, double* twiddle);
/* dft3d_generate_inverse_matrix: the inverse of the forward matrix of `nodes` (what DFT3D_INVERSE_SOLVE multiplies
 *   by), n*n complex doubles; *growth (may be NULL) receives max|M| * max|M^-1|. */
int dft3d_generate_inverse_matrix(long long n, const double* nodes, int nodes_on_output, double* matrix, double* growth);
int dft3d_generate_real_table(long long n, int sign, double scale, const double* nodes, int nodes_on_output,
                              float* hi, float* lo);

/*
 * The KDFT forward/inverse transform without any allocation (the paper has no counterpart to this call; it
 * exists for callers that cannot call cudaMalloc: code inside a section where the allocator is off limits,
 * plugins whose host owns all device memory, processes that have given every free byte to their own arena).
 *
 *   n0, n1, n2   sizes, each a multiple of 64, with n0*n1*n2 <= 2,097,152 points (the static scratch holds
 *                16 MiB); larger sizes return DFT3D_ERR_UNSUPPORTED and say so in error_message.
 *   w0, w1, w2   DEVICE pointers, 16-byte aligned: the per-axis real tables, [hi piece][lo piece], each piece
 *                (2*n_a)*(2*n_a) floats, exactly as dft3d_generate_real_table writes them (hi first, lo right
 *                after it).  Sign, inverse scaling and nonuniform nodes are whatever the caller generated.
 *   in, out      DEVICE pointers as for dft3d_execute (16-byte aligned, n0*n1*n2*8 bytes, not overlapping).
 *   cuda_stream  the stream the three axis kernels run on.
 *   error_message / error_message_size   optional HOST buffer that receives a description of a failure.
 *
 * The scratch cube between the axis passes is a file-scope device array inside the library: every GPU that
 * loads the library holds it until the process exits, every call on that GPU shares it, and it keeps the
 * previous call's contents (the call clears the one word that must start at zero).  Calls that overlap on the
 * same GPU, from any stream or thread, therefore race; run them one after the other.
 * The first call on a device resolves the array's address and sets kernel attributes; make that first call
 * before any stream capture.  Every call is synchronous: it enqueues its kernels, copies one status word back,
 * waits for the stream (cudaStreamSynchronize) and returns DFT3D_ERR_DEVICE_TIMEOUT if a kernel abandoned a wait.
 * It calls no cudaMalloc, cudaFree or other allocating routine.
 */
int dft3d_kdft_execute_static(long long n0, long long n1, long long n2, const float* w0, const float* w1,
                              const float* w2, const void* in, void* out, void* cuda_stream,
                              char* error_message, size_t error_message_size);

#ifdef __cplusplus
}
#endif
#endif /* DFT3D_H_ */
