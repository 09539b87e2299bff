/*
 * TEST INFRASTRUCTURE -- plain CPU eager evaluator for traced tensor ops.
 *
 * The LazyTensor paper (Section 3) states that a compiled IR graph must be
 * semantically equivalent to running the recorded operations individually.
 * This file *is* "running the operations individually": every function
 * evaluates exactly one traced op over whole arrays, into an output array the
 * caller allocated freshly for that op.  Nothing is fused, reordered, tiled or
 * reused between ops.
 *
 * The paper defines no numerics (its device code came from XLA); each op here
 * follows the textbook definition named in the comment above it:
 *   - + - * / sqrt            IEEE-754 binary32, round-to-nearest-even, one
 *                             rounding per op (build with -ffp-contract=off)
 *   - exp log tanh rsqrt ...  evaluated in binary64, rounded once to binary32
 *   - row_sum                 binary64 accumulation, left to right, one rounding
 *   - max/min/relu            NaN-propagating
 *   - bf16 nodes              operands widened to binary32, op in binary32,
 *                             result rounded to bf16 with ties-to-even
 *   - philox_bits             Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)
 *   - broadcast               operand index = output index with the operand's
 *                             size-1 (or missing leading) dimensions zeroed
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call this file.  It shares no code with the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_U8 = 2, ORC_I32 = 3, ORC_U32 = 4 };
enum { ORC_MAX_RANK = 6 };

typedef struct {
    void *data;
    int32_t dtype;
    int32_t rank;
    int64_t shape[ORC_MAX_RANK];
} orc_array;

enum {
    ORC_OK = 0,
    ORC_ERR_OP = 1,      /* unknown op name                          */
    ORC_ERR_DTYPE = 2,   /* dtype combination not defined for the op */
    ORC_ERR_SHAPE = 3    /* shapes do not broadcast / do not match   */
};

static int g_threads = 1;

void orc_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int orc_get_threads(void) { return g_threads; }

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ bf16 */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* Round binary32 to bfloat16, ties to even; NaN stays NaN (quiet bit set). */
static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16(f); }
float orc_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }

/* ------------------------------------------------------------ indexing */

static int64_t numel(const orc_array *a) {
    int64_t n = 1;
    for (int i = 0; i < a->rank; ++i) n *= a->shape[i];
    return n;
}

static int same_shape(const orc_array *a, const orc_array *b) {
    if (a->rank != b->rank) return 0;
    for (int i = 0; i < a->rank; ++i)
        if (a->shape[i] != b->shape[i]) return 0;
    return 1;
}

/* Can `a` be broadcast to `out` (dimensions aligned at the right)? */
static int broadcasts_to(const orc_array *a, const orc_array *out) {
    if (a->rank > out->rank) return 0;
    for (int i = 0; i < a->rank; ++i) {
        int64_t da = a->shape[a->rank - 1 - i];
        int64_t dout = out->shape[out->rank - 1 - i];
        if (da != dout && da != 1) return 0;
    }
    return 1;
}

/* Flat index into `a` of the element that output element `flat` reads. */
static int64_t bcast_index(const orc_array *a, const orc_array *out, int64_t flat) {
    int64_t idx = 0, stride = 1, rem = flat;
    for (int i = 0; i < out->rank; ++i) {
        int od = out->rank - 1 - i;
        int64_t coord = rem % out->shape[od];
        rem /= out->shape[od];
        int ad = a->rank - 1 - i;
        if (ad >= 0) {
            if (a->shape[ad] != 1) idx += coord * stride;
            stride *= a->shape[ad];
        }
    }
    return idx;
}

/* --------------------------------------------------- typed element access */

static float load_f(const orc_array *a, int64_t i) {
    return a->dtype == ORC_BF16 ? bf16_to_f32(((const uint16_t *)a->data)[i])
                                : ((const float *)a->data)[i];
}

static void store_f(orc_array *a, int64_t i, float v) {
    if (a->dtype == ORC_BF16) ((uint16_t *)a->data)[i] = f32_to_bf16(v);
    else ((float *)a->data)[i] = v;
}

static int is_float(int dt) { return dt == ORC_F32 || dt == ORC_BF16; }

/* -------------------------------------------------------- scalar kernels */

static float nan_f(void) { return nanf(""); }

static float max_nan(float a, float b) {
    if (a != a || b != b) return nan_f();
    return a > b ? a : b;
}

static float min_nan(float a, float b) {
    if (a != a || b != b) return nan_f();
    return a < b ? a : b;
}

enum { B_ADD, B_SUB, B_MUL, B_DIV, B_MAX, B_MIN, B_AND, B_OR, B_XOR, B_BAD };

static int binary_code(const char *op) {
    static const char *names[] = {"add", "sub", "mul", "div", "max", "min", "and", "or", "xor"};
    for (int i = 0; i < B_BAD; ++i)
        if (strcmp(op, names[i]) == 0) return i;
    return B_BAD;
}

static float binary_f32(int code, float a, float b) {
    switch (code) {
    case B_ADD: return a + b;
    case B_SUB: return a - b;
    case B_MUL: return a * b;
    case B_DIV: return a / b;
    case B_MAX: return max_nan(a, b);
    default:    return min_nan(a, b);
    }
}

/*
 * out = a (op) b, elementwise with broadcasting.
 * f32 / bf16: add sub mul div max min.  i32 / u32: add sub mul (wrapping),
 * max min, and or xor.  u8 (masks): and or xor.  All three arrays share one
 * dtype.
 */
int orc_binary(const char *op, const orc_array *a, const orc_array *b, orc_array *out) {
    int code = binary_code(op);
    if (code == B_BAD) return ORC_ERR_OP;
    if (a->dtype != out->dtype || b->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (!broadcasts_to(a, out) || !broadcasts_to(b, out)) return ORC_ERR_SHAPE;
    int dt = out->dtype;
    if (is_float(dt) && code > B_MIN) return ORC_ERR_DTYPE;
    if (dt == ORC_U8 && code < B_AND) return ORC_ERR_DTYPE;
    if ((dt == ORC_I32 || dt == ORC_U32) && code == B_DIV) return ORC_ERR_DTYPE;
    int64_t n = numel(out);
    int sa = same_shape(a, out), sb = same_shape(b, out);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t ia = sa ? i : bcast_index(a, out, i);
        int64_t ib = sb ? i : bcast_index(b, out, i);
        if (is_float(dt)) {
            store_f(out, i, binary_f32(code, load_f(a, ia), load_f(b, ib)));
        } else if (dt == ORC_U8) {
            uint8_t x = ((const uint8_t *)a->data)[ia], y = ((const uint8_t *)b->data)[ib];
            ((uint8_t *)out->data)[i] = code == B_AND ? (x & y) : code == B_OR ? (x | y) : (x ^ y);
        } else {
            uint32_t x = ((const uint32_t *)a->data)[ia], y = ((const uint32_t *)b->data)[ib], r;
            switch (code) {
            case B_ADD: r = x + y; break;
            case B_SUB: r = x - y; break;
            case B_MUL: r = x * y; break;
            case B_AND: r = x & y; break;
            case B_OR:  r = x | y; break;
            case B_XOR: r = x ^ y; break;
            case B_MAX:
                r = dt == ORC_I32 ? (uint32_t)((int32_t)x > (int32_t)y ? (int32_t)x : (int32_t)y)
                                  : (x > y ? x : y);
                break;
            default:
                r = dt == ORC_I32 ? (uint32_t)((int32_t)x < (int32_t)y ? (int32_t)x : (int32_t)y)
                                  : (x < y ? x : y);
                break;
            }
            ((uint32_t *)out->data)[i] = r;
        }
    }
    return ORC_OK;
}

enum { C_GT, C_GE, C_LT, C_LE, C_EQ, C_NE, C_BAD };

static int compare_code(const char *op) {
    static const char *names[] = {"gt", "ge", "lt", "le", "eq", "ne"};
    for (int i = 0; i < C_BAD; ++i)
        if (strcmp(op, names[i]) == 0) return i;
    return C_BAD;
}

#define CMP_BODY(x, y)                                     \
    (code == C_GT ? (x) > (y) : code == C_GE ? (x) >= (y)  \
     : code == C_LT ? (x) < (y) : code == C_LE ? (x) <= (y) \
     : code == C_EQ ? (x) == (y) : (x) != (y))

/* out (u8, 0 or 1) = a (cmp) b.  Float compares follow IEEE (NaN: only ne is true). */
int orc_compare(const char *op, const orc_array *a, const orc_array *b, orc_array *out) {
    int code = compare_code(op);
    if (code == C_BAD) return ORC_ERR_OP;
    if (a->dtype != b->dtype || out->dtype != ORC_U8) return ORC_ERR_DTYPE;
    if (!broadcasts_to(a, out) || !broadcasts_to(b, out)) return ORC_ERR_SHAPE;
    int dt = a->dtype;
    int64_t n = numel(out);
    int sa = same_shape(a, out), sb = same_shape(b, out);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t ia = sa ? i : bcast_index(a, out, i);
        int64_t ib = sb ? i : bcast_index(b, out, i);
        int r;
        if (is_float(dt)) {
            float x = load_f(a, ia), y = load_f(b, ib);
            r = CMP_BODY(x, y);
        } else if (dt == ORC_U8) {
            uint8_t x = ((const uint8_t *)a->data)[ia], y = ((const uint8_t *)b->data)[ib];
            r = CMP_BODY(x, y);
        } else if (dt == ORC_I32) {
            int32_t x = ((const int32_t *)a->data)[ia], y = ((const int32_t *)b->data)[ib];
            r = CMP_BODY(x, y);
        } else {
            uint32_t x = ((const uint32_t *)a->data)[ia], y = ((const uint32_t *)b->data)[ib];
            r = CMP_BODY(x, y);
        }
        ((uint8_t *)out->data)[i] = (uint8_t)(r ? 1 : 0);
    }
    return ORC_OK;
}

/* out = mask ? a : b.  mask is u8 (non-zero = true); a, b, out share a dtype. */
int orc_where(const orc_array *m, const orc_array *a, const orc_array *b, orc_array *out) {
    if (m->dtype != ORC_U8 || a->dtype != out->dtype || b->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (!broadcasts_to(m, out) || !broadcasts_to(a, out) || !broadcasts_to(b, out)) return ORC_ERR_SHAPE;
    int64_t n = numel(out);
    size_t es = out->dtype == ORC_BF16 ? 2 : out->dtype == ORC_U8 ? 1 : 4;
    int sm = same_shape(m, out), sa = same_shape(a, out), sb = same_shape(b, out);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t im = sm ? i : bcast_index(m, out, i);
        int64_t ia = sa ? i : bcast_index(a, out, i);
        int64_t ib = sb ? i : bcast_index(b, out, i);
        const char *src = ((const uint8_t *)m->data)[im] ? (const char *)a->data + ia * es
                                                        : (const char *)b->data + ib * es;
        memcpy((char *)out->data + i * es, src, es);
    }
    return ORC_OK;
}

enum {
    U_NEG, U_ABS, U_RELU, U_EXP, U_LOG, U_TANH, U_SQRT, U_RSQRT, U_RECIP, U_SQUARE,
    U_SIGMOID, U_GELU_TANH, U_NOT, U_BAD
};

static int unary_code(const char *op) {
    static const char *names[] = {"neg", "abs", "relu", "exp", "log", "tanh", "sqrt", "rsqrt",
                                  "recip", "square", "sigmoid", "gelu_tanh", "not"};
    for (int i = 0; i < U_BAD; ++i)
        if (strcmp(op, names[i]) == 0) return i;
    return U_BAD;
}

static float unary_f32(int code, float x) {
    double d = (double)x;
    switch (code) {
    case U_NEG:    return -x;
    case U_ABS:    return fabsf(x);
    case U_RELU:   return max_nan(x, 0.0f);
    case U_EXP:    return (float)exp(d);
    case U_LOG:    return (float)log(d);
    case U_TANH:   return (float)tanh(d);
    case U_SQRT:   return sqrtf(x);
    case U_RSQRT:  return (float)(1.0 / sqrt(d));
    case U_RECIP:  return (float)(1.0 / d);
    case U_SQUARE: return x * x;
    case U_SIGMOID:return (float)(1.0 / (1.0 + exp(-d)));
    default: {
        /* GELU, tanh form: 0.5 t (1 + tanh( sqrt(2/pi) (t + 0.044715 t^3) )) */
        double k = sqrt(2.0 / 3.14159265358979323846);
        return (float)(0.5 * d * (1.0 + tanh(k * (d + 0.044715 * d * d * d))));
    }
    }
}

/* out = f(a), same shape and dtype.  Float ops on f32/bf16; neg/abs also on i32; not on u8. */
int orc_unary(const char *op, const orc_array *a, orc_array *out) {
    int code = unary_code(op);
    if (code == U_BAD) return ORC_ERR_OP;
    if (a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (!same_shape(a, out)) return ORC_ERR_SHAPE;
    int dt = a->dtype;
    if (code == U_NOT) {
        if (dt != ORC_U8) return ORC_ERR_DTYPE;
    } else if (dt == ORC_I32) {
        if (code != U_NEG && code != U_ABS) return ORC_ERR_DTYPE;
    } else if (!is_float(dt)) {
        return ORC_ERR_DTYPE;
    }
    int64_t n = numel(out);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        if (code == U_NOT) {
            ((uint8_t *)out->data)[i] = ((const uint8_t *)a->data)[i] ? 0 : 1;
        } else if (dt == ORC_I32) {
            uint32_t x = ((const uint32_t *)a->data)[i];
            int neg = code == U_NEG || (int32_t)x < 0;
            ((uint32_t *)out->data)[i] = neg ? (0u - x) : x;
        } else {
            store_f(out, i, unary_f32(code, load_f(a, i)));
        }
    }
    return ORC_OK;
}

/*
 * Type conversion.  f32<->bf16 (RNE / exact); u8,i32,u32 -> f32 (value
 * conversion, RNE); f32 -> i32 truncates toward zero, saturates, NaN -> 0;
 * u8 -> i32/u32 zero-extends; i32 <-> u32 keeps the bit pattern;
 * f32/i32/u32 -> u8 yields (x != 0).
 */
int orc_convert(const orc_array *a, orc_array *out) {
    if (!same_shape(a, out)) return ORC_ERR_SHAPE;
    int64_t n = numel(out);
    int si = a->dtype, so = out->dtype;
    int ok = (is_float(si) && is_float(so)) || (so == ORC_F32 && !is_float(si)) ||
             (si == ORC_F32 && so == ORC_I32) || (si == ORC_U8 && (so == ORC_I32 || so == ORC_U32)) ||
             ((si == ORC_I32 || si == ORC_U32) && (so == ORC_I32 || so == ORC_U32)) ||
             (so == ORC_U8 && (si == ORC_F32 || si == ORC_I32 || si == ORC_U32 || si == ORC_U8));
    if (!ok) return ORC_ERR_DTYPE;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        if (is_float(si) && is_float(so)) {
            store_f(out, i, load_f(a, i));
        } else if (so == ORC_F32) {
            float v = si == ORC_U8 ? (float)((const uint8_t *)a->data)[i]
                    : si == ORC_I32 ? (float)((const int32_t *)a->data)[i]
                                    : (float)((const uint32_t *)a->data)[i];
            ((float *)out->data)[i] = v;
        } else if (si == ORC_F32 && so == ORC_I32) {
            float x = ((const float *)a->data)[i];
            int32_t r;
            if (x != x) r = 0;
            else if (x >= 2147483648.0f) r = INT32_MAX;
            else if (x <= -2147483648.0f) r = INT32_MIN;
            else r = (int32_t)x;
            ((int32_t *)out->data)[i] = r;
        } else if (so == ORC_U8) {
            int nz = si == ORC_F32 ? ((const float *)a->data)[i] != 0.0f
                   : si == ORC_U8 ? ((const uint8_t *)a->data)[i] != 0
                                  : ((const uint32_t *)a->data)[i] != 0;
            ((uint8_t *)out->data)[i] = (uint8_t)(nz ? 1 : 0);
        } else if (si == ORC_U8) {
            ((uint32_t *)out->data)[i] = ((const uint8_t *)a->data)[i];
        } else {
            ((uint32_t *)out->data)[i] = ((const uint32_t *)a->data)[i];
        }
    }
    return ORC_OK;
}

/* out (i32) = coordinate of each element along dimension `dim` of out's shape. */
int orc_iota(int dim, orc_array *out) {
    if (out->dtype != ORC_I32) return ORC_ERR_DTYPE;
    if (dim < 0 || dim >= out->rank) return ORC_ERR_SHAPE;
    int64_t n = numel(out);
    int64_t inner = 1;
    for (int d = dim + 1; d < out->rank; ++d) inner *= out->shape[d];
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i)
        ((int32_t *)out->data)[i] = (int32_t)((i / inner) % out->shape[dim]);
    return ORC_OK;
}

/*
 * Reductions over the other axes (the row reductions' siblings).
 * "col_*": reduce over every dimension but the last; `a` is viewed as
 * [rows, cols] with cols = its last extent, `out` has the same rank with all
 * leading extents 1.  "all_*": reduce over every element; `out` holds one element (rank 0 or [1]).
 * Sums accumulate in binary64 in index order and round once; max / min
 * propagate NaN.  Float dtypes only.
 */
static int reduce_kind(const char *op, const char *prefix) {
    size_t n = strlen(prefix);
    if (strncmp(op, prefix, n) != 0) return -1;
    return strcmp(op + n, "sum") == 0 ? 0 : strcmp(op + n, "max") == 0 ? 1 : strcmp(op + n, "min") == 0 ? 2 : -1;
}

int orc_col_reduce(const char *op, const orc_array *a, orc_array *out) {
    int kind = reduce_kind(op, "col_");
    if (kind < 0) return ORC_ERR_OP;
    if (!is_float(a->dtype) || a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (a->rank < 1 || out->rank != a->rank || out->shape[a->rank - 1] != a->shape[a->rank - 1]) return ORC_ERR_SHAPE;
    for (int d = 0; d + 1 < a->rank; ++d)
        if (out->shape[d] != 1) return ORC_ERR_SHAPE;
    int64_t cols = a->shape[a->rank - 1];
    int64_t rows = cols ? numel(a) / cols : 0;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t c = 0; c < cols; ++c) {
        float res;
        if (kind == 0) {
            double acc = 0.0;
            for (int64_t r = 0; r < rows; ++r) acc += (double)load_f(a, r * cols + c);
            res = (float)acc;
        } else {
            res = kind == 1 ? -INFINITY : INFINITY;
            for (int64_t r = 0; r < rows; ++r) {
                float x = load_f(a, r * cols + c);
                res = kind == 1 ? max_nan(res, x) : min_nan(res, x);
            }
        }
        store_f(out, c, res);
    }
    return ORC_OK;
}

int orc_all_reduce(const char *op, const orc_array *a, orc_array *out) {
    int kind = reduce_kind(op, "all_");
    if (kind < 0) return ORC_ERR_OP;
    if (!is_float(a->dtype) || a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (out->rank > 1 || numel(out) != 1) return ORC_ERR_SHAPE;
    int64_t n = numel(a);
    float res;
    if (kind == 0) {
        double acc = 0.0;
        for (int64_t i = 0; i < n; ++i) acc += (double)load_f(a, i);
        res = (float)acc;
    } else {
        res = kind == 1 ? -INFINITY : INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            float x = load_f(a, i);
            res = kind == 1 ? max_nan(res, x) : min_nan(res, x);
        }
    }
    store_f(out, 0, res);
    return ORC_OK;
}

/* ------------------------------------------------------------------ views */

static size_t elem_size(int dt) { return dt == ORC_BF16 ? 2 : dt == ORC_U8 ? 1 : 4; }

/* Row-major strides (in elements) of `a`. */
static void strides_of(const orc_array *a, int64_t *st) {
    int64_t s = 1;
    for (int d = a->rank - 1; d >= 0; --d) {
        st[d] = s;
        s *= a->shape[d];
    }
}

/* Coordinates of flat index i in an array of `rank` dimensions `shape`. */
static void unravel(int64_t i, const int64_t *shape, int rank, int64_t *idx) {
    for (int d = rank - 1; d >= 0; --d) {
        idx[d] = shape[d] ? i % shape[d] : 0;
        i = shape[d] ? i / shape[d] : 0;
    }
}

/* out = a with another shape of the same element count; element order (row-major) is kept. */
int orc_reshape(const orc_array *a, orc_array *out) {
    if (a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (numel(a) != numel(out)) return ORC_ERR_SHAPE;
    memcpy(out->data, a->data, (size_t)numel(a) * elem_size(a->dtype));
    return ORC_OK;
}

/* out[.., k, ..] = a[.., start + k, ..] along dimension `dim`; out's extent there is the slice length. */
int orc_narrow(const orc_array *a, int dim, int64_t start, orc_array *out) {
    if (a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (a->rank != out->rank || dim < 0 || dim >= a->rank) return ORC_ERR_SHAPE;
    for (int d = 0; d < a->rank; ++d)
        if (d != dim && a->shape[d] != out->shape[d]) return ORC_ERR_SHAPE;
    if (start < 0 || start + out->shape[dim] > a->shape[dim]) return ORC_ERR_SHAPE;
    int64_t st[ORC_MAX_RANK], idx[ORC_MAX_RANK];
    strides_of(a, st);
    size_t es = elem_size(a->dtype);
    int64_t n = numel(out);
    for (int64_t i = 0; i < n; ++i) {
        unravel(i, out->shape, out->rank, idx);
        idx[dim] += start;
        int64_t src = 0;
        for (int d = 0; d < a->rank; ++d) src += idx[d] * st[d];
        memcpy((char *)out->data + (size_t)i * es, (const char *)a->data + (size_t)src * es, es);
    }
    return ORC_OK;
}

/* out dimension i is a's dimension perm[i]: out[j0, j1, ..] = a[i0, i1, ..] with i[perm[k]] = j[k]. */
int orc_permute(const orc_array *a, const int *perm, orc_array *out) {
    if (a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (a->rank != out->rank) return ORC_ERR_SHAPE;
    int seen[ORC_MAX_RANK] = {0};
    for (int k = 0; k < a->rank; ++k) {
        if (perm[k] < 0 || perm[k] >= a->rank || seen[perm[k]]) return ORC_ERR_SHAPE;
        seen[perm[k]] = 1;
        if (out->shape[k] != a->shape[perm[k]]) return ORC_ERR_SHAPE;
    }
    int64_t st[ORC_MAX_RANK], idx[ORC_MAX_RANK];
    strides_of(a, st);
    size_t es = elem_size(a->dtype);
    int64_t n = numel(out);
    for (int64_t i = 0; i < n; ++i) {
        unravel(i, out->shape, out->rank, idx);
        int64_t src = 0;
        for (int k = 0; k < a->rank; ++k) src += idx[k] * st[perm[k]];
        memcpy((char *)out->data + (size_t)i * es, (const char *)a->data + (size_t)src * es, es);
    }
    return ORC_OK;
}

/* out = base with the slice [start, start + upd.shape[dim]) along `dim` replaced by upd. */
int orc_update_slice(const orc_array *base, const orc_array *upd, int dim, int64_t start, orc_array *out) {
    if (base->dtype != out->dtype || upd->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (!same_shape(base, out) || upd->rank != base->rank || dim < 0 || dim >= base->rank) return ORC_ERR_SHAPE;
    for (int d = 0; d < base->rank; ++d)
        if (d != dim && upd->shape[d] != base->shape[d]) return ORC_ERR_SHAPE;
    if (start < 0 || start + upd->shape[dim] > base->shape[dim]) return ORC_ERR_SHAPE;
    size_t es = elem_size(out->dtype);
    memcpy(out->data, base->data, (size_t)numel(base) * es);
    int64_t st[ORC_MAX_RANK], idx[ORC_MAX_RANK];
    strides_of(out, st);
    int64_t n = numel(upd);
    for (int64_t i = 0; i < n; ++i) {
        unravel(i, upd->shape, upd->rank, idx);
        idx[dim] += start;
        int64_t dst = 0;
        for (int d = 0; d < out->rank; ++d) dst += idx[d] * st[d];
        memcpy((char *)out->data + (size_t)dst * es, (const char *)upd->data + (size_t)i * es, es);
    }
    return ORC_OK;
}

/* ---------------------------------------------------------------- Philox */

/*
 * One Philox4x32 block with 10 rounds (Salmon et al., SC'11, Section 3.3 /
 * Table 2): each round multiplies two counter words by fixed odd constants,
 * swaps high and low halves across the lanes and folds in the key; the key is
 * advanced by the Weyl constants between rounds.
 */
static void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0;
        k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    philox4x32_10(ctr, key, out);
}

/*
 * out (u32): element with flat index i takes word (i mod 4) of the block whose
 * counter is (lo32(q), hi32(q), lo32(offset), hi32(offset)), q = floor(i / 4),
 * under the key (lo32(seed), hi32(seed)).
 */
int orc_philox_bits(uint64_t seed, uint64_t offset, orc_array *out) {
    if (out->dtype != ORC_U32) return ORC_ERR_DTYPE;
    int64_t n = numel(out);
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        uint64_t q = (uint64_t)i / 4;
        uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), (uint32_t)offset, (uint32_t)(offset >> 32)};
        uint32_t w[4];
        philox4x32_10(ctr, key, w);
        ((uint32_t *)out->data)[i] = w[i % 4];
    }
    return ORC_OK;
}

/* ------------------------------------------------------- row reductions */

/*
 * Reduce over the last dimension, keeping it with extent 1.
 * "row_sum": binary64 accumulation left to right, one rounding to the output
 * type.  "row_max" / "row_min": NaN-propagating.  Float dtypes only.
 */
int orc_row_reduce(const char *op, const orc_array *a, orc_array *out) {
    int kind = strcmp(op, "row_sum") == 0 ? 0 : strcmp(op, "row_max") == 0 ? 1
             : strcmp(op, "row_min") == 0 ? 2 : -1;
    if (kind < 0) return ORC_ERR_OP;
    if (!is_float(a->dtype) || a->dtype != out->dtype) return ORC_ERR_DTYPE;
    if (a->rank < 1 || out->rank != a->rank || out->shape[a->rank - 1] != 1) return ORC_ERR_SHAPE;
    for (int d = 0; d + 1 < a->rank; ++d)
        if (a->shape[d] != out->shape[d]) return ORC_ERR_SHAPE;
    int64_t cols = a->shape[a->rank - 1];
    int64_t rows = numel(out);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        float res;
        if (kind == 0) {
            double acc = 0.0;
            for (int64_t c = 0; c < cols; ++c) acc += (double)load_f(a, r * cols + c);
            res = (float)acc;
        } else {
            res = kind == 1 ? -INFINITY : INFINITY;
            for (int64_t c = 0; c < cols; ++c) {
                float x = load_f(a, r * cols + c);
                res = kind == 1 ? max_nan(res, x) : min_nan(res, x);
            }
        }
        store_f(out, r, res);
    }
    return ORC_OK;
}
