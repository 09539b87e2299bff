// Register-program virtual machine shared by the planner (host) and the kernels (device).
//
// A fusion group runs as one kernel in which every thread owns a chunk of LT_VM_V
// consecutive elements of a row and interprets the group's program on them.  The
// machine is an accumulator machine: ACC plus LT_VM_NT temporaries, each LT_VM_V
// 32-bit lanes wide (f32 values, or i32/u32/u8 values held as integers).  Every
// (operation, operand source) pair has its own opcode so that one warp-uniform jump
// reaches straight-line code that names its registers statically -- a register file
// indexed at run time would live in local memory.
#pragma once
#ifdef __CUDACC_RTC__
// the run-time compiler has no standard headers: the fixed-width names this file and the shells use
typedef unsigned char uint8_t;
typedef unsigned short uint16_t;
typedef unsigned int uint32_t;
typedef unsigned long long uint64_t;
typedef int int32_t;
typedef long long int64_t;
#else
#include <stdint.h>
#endif

#define LT_VM_V 8          // lanes per chunk
#define LT_EW_THREADS 256  // CTA size of the elementwise and multi-tensor kernels
#define LT_VM_NT 3         // temporaries T0..T2 (a fourth one costs 8 registers per thread, i.e. a resident block per SM)
#define LT_VM_ND 4         // load destinations: the temporaries, then ACC
#define LT_VM_NSRC 4       // operand sources of two-operand opcodes: the temporaries, then S (broadcast immediate)
#define LT_VM_SRC_S 3
#define LT_VM_MAX_INS 118     // the program is followed by an END and one padding slot
#define LT_VM_MAX_PTR 12
#define LT_VM_MAX_SCAL 32
// byte offsets inside the per-CTA shared-memory block the PTX core reads (struct Staged in kernels.cu)
#define LT_VM_SM_SCAL 960   // immediates, after (LT_VM_MAX_INS + 2) instruction words
#define LT_VM_SM_PTR 1088   // pointer table
#define LT_VM_SM_SOFF 1184  // per-slot offset inside a staging buffer, or 0xFFFFFFFF
#define LT_VM_SM_LOOP 1232  // struct LtLoop: constants of the chunk loop the PTX core runs by itself
#define LT_VM_SM_STG 1296   // LtLoop::stg, the list of inputs staged by asynchronous copies
#define LT_VM_SM_RED 1520   // 64 floats: cross-warp exchange of the row reductions (two alternating halves)
#define LT_VM_STAGE_PIECE 4096  // bytes one 16-byte piece of a staged input takes per stage (256 threads x 16)

#define LT_MULTI_MAX_INS 64
#define LT_MULTI_MAX_INST 384   // instances (tensors) per multi-tensor launch
#define LT_MULTI_MAX_PTRS 2816  // pointer-table entries per launch (instances x slots)
#define LT_MULTI_MAX_SLOTS 8
#define LT_MULTI_SUB 8          // chunks each thread runs per super-chunk

struct LtIns {
    uint32_t op;
    uint32_t imm;  // pointer slot or immediate slot
};

// element classes of a pointer slot relative to the group's [rows, cols] domain
// LT_CLS_PITCHED: a full-class operand whose rows lie `pitch` elements apart (a slice of wider rows, read in place)
enum { LT_CLS_FULL = 0, LT_CLS_COLVEC = 1, LT_CLS_ROWVEC = 2, LT_CLS_SCALAR = 3, LT_CLS_PITCHED = 4 };
// LT_CLS_REDUCED + 3 * axis + kind: a store slot of an elementwise program whose value is not written but reduced --
// over the rows of every column (axis 0) or over everything (axis 1); kind 0 sum, 1 max, 2 min -- into binary64
// partial results that a second, small kernel finishes (compiled shells only)
enum { LT_CLS_REDUCED = 8 };
// storage dtypes (same numbering as lt_dtype)
enum { LT_ST_F32 = 0, LT_ST_BF16 = 1, LT_ST_U8 = 2, LT_ST_I32 = 3, LT_ST_U32 = 4 };

enum { F2_ADD = 0, F2_SUB, F2_RSUB, F2_MUL, F2_DIV, F2_RDIV, F2_MAX, F2_MIN, F2_COUNT };
enum { I2_ADD = 0, I2_SUB, I2_RSUB, I2_MUL, I2_AND, I2_OR, I2_XOR, I2_MAXS, I2_MINS, I2_MAXU, I2_MINU, I2_COUNT };
// compare index = type * 6 + cc ; type 0 f32, 1 signed, 2 unsigned ; cc: GT GE LT LE EQ NE
enum { CC_GT = 0, CC_GE, CC_LT, CC_LE, CC_EQ, CC_NE };
enum { CMP_COUNT = 18 };
enum { F2M_ADD = 0, F2M_SUB, F2M_RSUB, F2M_MUL, F2M_COUNT };

enum {
    OP_END = 0,
    OP_MOV_T_ACC = 1,                        // +k : T[k] = ACC
    OP_MOV_ACC_T = OP_MOV_T_ACC + LT_VM_NT,  // +k : ACC = T[k]
    OP_MOV_ACC_S = OP_MOV_ACC_T + LT_VM_NT,  // ACC = broadcast(imm slot)
    OP_ST = 20,          // store ACC to pointer slot imm, any class and dtype (handled outside the PTX core)
    OP_IOTA_COL = 21,    // ACC = column index of each lane (i32)
    OP_IOTA_ROW = 22,    // ACC = (row / scal[imm]) % scal[imm+1] (i32), same in every lane
    OP_PHILOX = 23,      // ACC = random bits of each lane's flat index; scal[imm..imm+3] = seed lo,hi, offset lo,hi
    OP_RED_SUM = 24,     // ACC = sum over the row, broadcast to every lane   (row kernel only)
    OP_RED_MAX = 25,
    OP_RED_MIN = 26,
    // one-operand ops on ACC
    OP_U_NEG = 30, OP_U_ABS, OP_U_RELU, OP_U_EXP, OP_U_LOG, OP_U_TANH, OP_U_SQRT, OP_U_RSQRT, OP_U_RECIP,
    OP_U_SQUARE, OP_U_SIGMOID, OP_U_GELU, OP_U_RBF16 /* round to bf16, keep as f32 */,
    OP_U_INEG = 43, OP_U_IABS = 44, OP_U_NOT = 45,
    OP_C_I2F = 46, OP_C_U2F = 47, OP_C_F2I = 48, OP_C_NZF = 49 /* f32 != 0 -> 0/1 */, OP_C_NZI = 50,
    // Loads deliver widened 32-bit lanes.  The planner emits the generic forms OP_LD / OP_F2M / OP_ST with
    // the pointer slot as immediate; when a kernel starts, each is rewritten ("linked") for this launch's
    // pointers into a vector-path opcode the PTX core executes itself -- ...G: 128-bit global access,
    // ...S: read from the thread's staging buffer (immediate = byte offset in the buffer).  Slots that
    // cannot use vector accesses keep the generic opcode, which the C++ around the core handles.
    // size 0/1/2 = 4/2/1-byte elements; class 0 = full, 1 = column vector; d < LT_VM_NT = T[d], else ACC.
    OP_LD = 51,                              // +d
    OP_LDG = OP_LD + LT_VM_ND,               // +(size * 2 + class) * LT_VM_ND + d
    OP_LDS = OP_LDG + 6 * LT_VM_ND,          // +size * LT_VM_ND + d : staged load
    OP_STG = OP_LDS + 3 * LT_VM_ND,          // +size : vector store of ACC to a full-class slot
    OP_F2M = OP_STG + 3,                     // +k : ACC = ACC (op) widened chunk of slot imm; k: see F2M_*
    OP_F2MG = OP_F2M + F2M_COUNT,            // +(k * 3 + size) * 2 + class
    OP_F2MS = OP_F2MG + F2M_COUNT * 6,       // +k * 3 + size
    // two-operand families: opcode = base + index * LT_VM_NSRC + source
    OP_F2 = OP_F2MS + F2M_COUNT * 3,         // ACC = ACC (op) src, f32: see F2_*
    OP_I2 = OP_F2 + F2_COUNT * LT_VM_NSRC,   // integer: see I2_*
    OP_CMP = OP_I2 + I2_COUNT * LT_VM_NSRC,  // ACC = (ACC cmp src) ? 1 : 0 : see CC_*
    OP_WHERE_A = OP_CMP + CMP_COUNT * LT_VM_NSRC,     // + m * LT_VM_NSRC + src : ACC = T[m] != 0 ? ACC : src
    OP_WHERE_B = OP_WHERE_A + LT_VM_NT * LT_VM_NSRC,  // + m * LT_VM_NSRC + src : ACC = T[m] != 0 ? src : ACC
    OP_LIMIT = OP_WHERE_B + LT_VM_NT * LT_VM_NSRC
};
static_assert(OP_MOV_ACC_S < OP_ST && OP_C_NZI < OP_LD, "opcode map");

// Per-CTA constants of the chunk loop, in shared memory (read by the PTX core with broadcast loads).
struct LtLoop {
    uint32_t stride, n_chunks, body_off, depth;          // chunks between a thread's iterations; total; byte offset of the per-chunk part of the program; staging depth
    // one staging buffer; all of them; shared address of the first; inloop bits 0-1: the core loops by itself, 1 = over
    // chunks recomputing coordinates, 2 = a fixed distance ahead with unchanged columns; bit 8 = L2 prefetch on
    uint32_t buf_bytes, buf_total, stage_base, inloop;
    uint32_t rowcol, cpr, div_mul, div_sh1;
    // stg_n: staged inputs by element size, 4-byte | 2-byte << 8 | 1-byte << 16 (the list is sorted that way)
    uint32_t div_sh2, cols, prefetch, stg_n;             // prefetch: 1 = L2-prefetch the next chunk of full-class loads
    struct {
        uint32_t ptr_lo, ptr_hi, dst, shift;             // source pointer, offset inside a staging buffer, log2(element bytes)
    } stg[LT_VM_MAX_PTR];
    uint32_t pf_lo, pf_hi;                               // byte distance (4-byte elements) between a thread's iterations
    uint32_t n4_lo, n4_hi;                               // 4 * number of elements
    uint32_t group, inline_rows;                         // row kernel: threads per row; 1 = reductions / row index / random bits run in the core
    uint32_t dpf_lo, dpf_hi;                             // depth * pf: distance to the chunk whose inputs are staged next
};

// Kernel parameter block of the elementwise and row-reduction kernels.  It is passed by
// value as a __grid_constant__ kernel parameter, so program, pointers and immediates are
// read from the constant bank with no separate upload.
struct LtKParams {
    uint64_t ptr[LT_VM_MAX_PTR];
    uint32_t scal[LT_VM_MAX_SCAL];
    LtIns ins[LT_VM_MAX_INS];
    uint8_t io_dtype[LT_VM_MAX_PTR];
    uint8_t io_class[LT_VM_MAX_PTR];
    uint8_t io_stage[LT_VM_MAX_PTR];  // first 16-byte piece of the slot in a staging buffer, 0xFF = not staged
    uint32_t pitch[LT_VM_MAX_PTR];    // LT_CLS_PITCHED slots: elements between the starts of consecutive rows
    uint32_t stage_depth;   // staging buffers per thread (0 = loads go straight to registers)
    uint32_t stage_pieces;  // 16-byte pieces per staging buffer
    uint32_t n_ins;
    uint32_t n_pro;         // leading instructions run once per thread; the chunk loop restarts after them
    uint32_t rowcol;        // 0: flat chunks over n elements; 1: chunks stay inside rows
    uint64_t n;             // rows * cols
    uint32_t rows, cols;    // rowcol only
    uint32_t cpr;           // chunks per row = ceil(cols / V)
    uint32_t div_mul, div_sh1, div_sh2;  // row = chunk / cpr without a divide
    uint64_t n_chunks;
    // row kernel geometry
    uint32_t group;         // threads per row (power of two)
    uint32_t group_log2;
    uint32_t rows_per_cta;
};

// Parameter block of the multi-tensor kernel: one program, many instances.
struct LtMultiParams {
    LtIns ins[LT_MULTI_MAX_INS];
    uint32_t scal[LT_VM_MAX_SCAL];
    uint8_t io_dtype[LT_VM_MAX_PTR];
    uint8_t io_stage[LT_VM_MAX_PTR];               // first staging piece of the slot, 0xFF = not staged (same for all instances)
    uint32_t stage_depth, stage_pieces;
    uint32_t n_ins;
    uint32_t n_inst;
    uint32_t n_slots;
    uint32_t total_super;                          // total super-chunks
    uint32_t super_prefix[LT_MULTI_MAX_INST + 1];  // super-chunks before instance i
    uint32_t numel[LT_MULTI_MAX_INST];
    uint64_t ptr[LT_MULTI_MAX_PTRS];               // [instance * n_slots + slot]
};
