/* mom.h -- C ABI of the B200 Linnea-equation library.
 *
 * A Linnea equation (paper Section 2, "Operations": an Equation is a bag of variadic Mul / Add ops
 * whose Yield is one result) is restricted here to
 *
 *        X = M1 * M2 * ... * Mn  +  T1 + ... + Tk          (n >= 1, k >= 0)
 *
 * over f32 matrices that each carry one compile-time property (paper Section 2, "Matrix Attribute"
 * and "Types": a Matrix type is a property, a static [rows, cols] and an element type; Identity is
 * its own type).  Planning applies the paper's three transformations (Section 2, "Transformations"):
 * identity simplification (A*I -> A, I*I -> I), matrix-chain reordering that minimises the number of
 * useful scalar multiplications taking properties into account, and property propagation that gives
 * every intermediate and the result a concrete type.  Execution runs each binary product with a
 * property-specialised sm_100a kernel and fuses the Add terms into the last product.
 *
 * Conventions
 *   - Every function returns mom_status_t (except mom_status_string); nothing throws.  Output arguments
 *     are written only on MOM_OK unless stated otherwise.
 *   - State.  Planning is a pure function of its arguments and may run from any number of threads at
 *     once.  The library keeps two pieces of process-wide state, both per GPU and both behind a mutex:
 *     a table of hardware facts and one-time kernel settings (SM count, shared-memory limits raised with
 *     cudaFuncSetAttribute), filled when a device is first used, so one process may run plans on several
 *     GPUs; and the fixed scratch array of mom_product_3xtf32_noalloc.  A plan's parenthesization, steps and
 *     sizes never change after creation; the plan also owns launcher state (tile tables, a status word,
 *     timing events, copy streams) that is created at its first execute on a device and rebuilt if the plan
 *     is later executed on another device.  The execute calls take a per-plan lock while they enqueue, so
 *     several threads may execute one plan (on one device); mom_plan_last_launch_count, the step timers and
 *     mom_plan_device_status then describe whichever call came last.  A plan must not be destroyed while
 *     another thread is inside a call on it.
 *   - "host" / "device" below says which address space a pointer must belong to.
 *   - Matrix storage (device): dense row-major f32, leading dimension == cols, base address aligned
 *     to 16 bytes.  Entries outside a triangular operand's structure must be stored as zeros (paper
 *     Section 2: the property dictates how the buffer is filled); the library relies on this and
 *     does not check it.  Identity operands have no storage: their pointer may be NULL and is never
 *     dereferenced.
 *   - The result X is always written as a full dense rows x cols matrix; entries outside the
 *     result's inferred structure are written as +0.0f.  X must not alias any input or the workspace.
 *   - Execution is asynchronous on the given stream.  All argument errors are reported before
 *     anything is enqueued (mom_equation_execute_host included: no copy from the caller's buffers
 *     starts before its arguments have been checked, and if a CUDA call fails later it waits for the copies
 *     already enqueued before it returns the error).
 */
#ifndef MOM_H_
#define MOM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOM_OK = 0,
    MOM_ERR_INVALID_ARG = 1,         /* null pointer, n_chain < 1, rows/cols < 1, bad enum, batch < 1 */
    MOM_ERR_PROPERTY = 2,            /* triangular, Diagonal, Symmetric or Identity descriptor that is not square */
    MOM_ERR_DTYPE = 3,               /* element type other than f32                                   */
    MOM_ERR_SHAPE_MISMATCH = 4,      /* inner dimensions differ, or an Add term's shape != X's shape  */
    MOM_ERR_OVERFLOW = 5,            /* a multiplication count does not fit in 63 bits                */
    MOM_ERR_ALLOC = 6,               /* host or (first execute only) device allocation failed         */
    MOM_ERR_WORKSPACE_TOO_SMALL = 7,
    MOM_ERR_ALIGNMENT = 8,           /* a device pointer is not 16-byte aligned                       */
    MOM_ERR_ARCH = 9,                /* the current device is not sm_100                              */
    MOM_ERR_CUDA = 10,               /* a CUDA runtime / driver call failed                           */
    MOM_ERR_DEVICE_TIMEOUT = 11,     /* a bounded device-side wait expired (see mom_plan_device_status) */
    MOM_ERR_BUFFER_TOO_SMALL = 12,   /* string buffer too small; `needed` tells the size              */
    MOM_ERR_LIMIT = 13               /* size beyond a documented fixed maximum                        */
} mom_status_t;

/* Paper Section 2, "Matrix Attribute" / "Types".  Triangles are non-strict and non-unit: the diagonal
 * is an ordinary stored entry (Listing 2 fills the diagonal with the fill value).
 * MOM_DIAGONAL is one of the further properties the paper's conclusion announces (it prints no rule for
 * it): a square matrix, stored densely like every other operand, whose entries off the diagonal are zeros.
 * Unlike Identity its diagonal is data: it is never simplified away, D*A costs one multiplication per
 * structural entry of A and runs as a scaling pass, D^T = D, and the lattice of product and sum types is
 * Identity < Diagonal < {lowerTri, upperTri} < general.
 * MOM_SYMMETRIC is another such property: a square matrix stored densely IN FULL (both triangles) with
 * a_ij = a_ji; the library relies on that and does not check it.  Its structure is full, so it costs what a
 * general matrix costs; S^T = S; a product with a Symmetric factor is general; a sum of Symmetric, Diagonal
 * and Identity summands is Symmetric.  Symmetric values also arise inside plans: where factor names are known
 * (mom_equation_plan_sum with names, mom_expression_plan), a sub-chain that reads Y * Y^T factor by factor
 * is typed Symmetric, and the tree that splits it in the middle computes Y once and then only the lower
 * triangle of Y * Y^T (MOM_KIND_GRAM): the right half is never multiplied.  A computed Symmetric value is
 * symmetric up to rounding in its diagonal blocks and exactly symmetric elsewhere (mirrored).
 * MOM_STRICT_LOWER / MOM_STRICT_UPPER and MOM_UNIT_LOWER / MOM_UNIT_UPPER are two more such properties: square
 * triangular matrices, stored densely, whose diagonal holds zeros (strict) or ones (unit; stored as 1.0f, the
 * library relies on that and does not check it).  An entry known to be 1 needs no multiplication, as with
 * Identity: a multiplication counts only when both entries are structural non-zeros and neither is a known 1,
 * so a unit triangle costs what the strict one costs.  Within one orientation the diagonal of a product is the
 * product of the diagonals (strict if either factor is strict, unit if both are unit); in a sum the diagonals add
 * (strict + strict = strict, strict + unit or Identity = unit, anything else an ordinary triangle); the transpose
 * swaps lower and upper and keeps the kind.  The kernels treat them as the enclosing ordinary triangle: a strict
 * result's diagonal is computed as a sum of products with an exact zero factor (+0 for finite inputs), a unit
 * result's diagonal as 1*1 plus such zeros (exactly 1). */
typedef enum { MOM_GENERAL = 0, MOM_LOWER_TRI = 1, MOM_UPPER_TRI = 2, MOM_IDENTITY = 3, MOM_DIAGONAL = 4, MOM_SYMMETRIC = 5,
               MOM_STRICT_LOWER = 6, MOM_STRICT_UPPER = 7, MOM_UNIT_LOWER = 8, MOM_UNIT_UPPER = 9 } mom_property_t;
typedef enum { MOM_F32 = 0 } mom_dtype_t;

/* Arithmetic used by the product kernels.
 *   MOM_VARIANT_3XTF32: tensor-core MMA (kind::tf32 / .tf32) on operands split as a = hi + lo,
 *       accumulating lo*hi + hi*lo + hi*hi in f32 (f32-level accuracy).  Three kernels, chosen by size:
 *       large products (m*n*k >= 6 * 2^26 that the kernel below does not take) whose leading
 *       dimensions TMA can address (multiples of 4 elements) run on the tcgen05 kernel that takes its operands as
 *       hi / lo planes (a pre-pass writes them; TMA, tensor memory, persistent CTAs); products of operands
 *       whose stored rows are 16-byte addressable (transposed ones included) with a result of at least
 *       65536 entries and 6 * 10^7 <= m*n*k < 10^9, or
 *       m*n*k < 4 * 10^9 with at most 148 result tiles of 128 x 128, or (an equation of one product only)
 *       m*n*k < 10^10 with at most 74 result tiles of 256 x 256 (CTA pairs), run on the tcgen05 kernel that reads the
 *       operands as stored and splits them on the way into shared and tensor memory (one launch); everything
 *       else runs on the warp-level kernel (mma.sync on the operands as stored, one launch).  A plan with packed
 *       operands or a packed result keeps its large products on the first kernel, which addresses the containers in place.
 *   MOM_VARIANT_FFMA: plain f32 fused multiply-add on CUDA cores.
 *   MOM_VARIANT_3XTF32_FORCE: every TMA-addressable product runs on the tcgen05 kernel, the others on
 *       the FFMA kernel; meant for testing the tcgen05 kernel on small shapes.
 *   MOM_VARIANT_3XTF32_WARP: every product runs on the warp-level kernel; meant for testing it on
 *       large shapes.
 *   MOM_VARIANT_3XTF32_INLINE: every product the in-kernel-split tcgen05 kernel takes runs there, whatever its
 *       size, the others on the warp-level kernel; meant for testing.
 * Whatever the variant, equations small enough for shared memory run as one fused launch, and products
 * with a Diagonal factor run on the scaling kernel. */
typedef enum { MOM_VARIANT_3XTF32 = 0, MOM_VARIANT_FFMA = 1, MOM_VARIANT_3XTF32_FORCE = 2, MOM_VARIANT_3XTF32_WARP = 3,
               MOM_VARIANT_3XTF32_INLINE = 4 } mom_variant_t;

/* Kind of a binary product, by which operands are triangular. */
typedef enum {
    MOM_KIND_GG = 0,     /* general * general                                  */
    MOM_KIND_TG = 1,     /* triangular * general                               */
    MOM_KIND_GT = 2,     /* general * triangular                               */
    MOM_KIND_TT = 3,     /* L*L or U*U: result keeps the triangle              */
    MOM_KIND_TTMIX = 4,  /* L*U or U*L: result is general                      */
    MOM_KIND_SCALE = 5,  /* a Diagonal operand on either side: rows or columns of the other operand are scaled */
    MOM_KIND_GRAM = 6    /* Y * Y^T: rhs is the same value as lhs, read transposed; useful_mults counts entries i >= j */
} mom_kind_t;

typedef struct {
    int64_t rows, cols;
    int32_t property;    /* mom_property_t */
    int32_t dtype;       /* mom_dtype_t    */
} mom_matrix_desc_t;

/* One binary product of the plan.  Ids: 0..n_chain-1 are the original chain operands, n_chain.. are
 * intermediates in the order they are produced; the last step's `out` is the chain's value. */
typedef struct {
    int32_t lhs, rhs, out;
    int32_t kind;                    /* mom_kind_t */
    int32_t lhs_property, rhs_property, out_property;
    int32_t uses_tensor_cores;       /* 1: tcgen05 3xTF32 kernel on operand planes, 3: tcgen05 3xTF32 kernel splitting in shared memory,
                                        2: warp-level 3xTF32 kernel, 0: FFMA kernel (MOM_KIND_SCALE: the scaling kernel) */
    int32_t lhs_transposed, rhs_transposed;   /* the operand is read transposed (an original chain operand used transposed; the rhs of MOM_KIND_GRAM) */
    int64_t m, n, k;                 /* out is m x n, contraction length k */
    uint64_t useful_mults;           /* scalar multiplications with both factors structurally non-zero */
} mom_step_t;

typedef struct mom_plan mom_plan_t;          /* opaque; host memory; what was planned never changes (see "State" above) */
typedef struct CUstream_st *mom_stream_t;    /* a CUDA stream handle (cudaStream_t) */

/* Fill a descriptor (paper Section 2, "Types": property, static shape, element type).
 * Errors: INVALID_ARG (out NULL, rows/cols < 1, unknown property), PROPERTY (non-square triangular or
 * Identity), DTYPE, LIMIT (rows or cols above 2^31 - 1025: the kernels index with 32-bit integers). */
mom_status_t mom_matrix_desc(int64_t rows, int64_t cols, mom_property_t property, mom_dtype_t dtype,
                             mom_matrix_desc_t *out /* host */);

/* Column-slab split of one equation over `world` devices (paper Section 5 names non-rectangular iteration spaces and
 * other containers as future work; this is the data-parallel split that needs neither).  Column j of
 * X = M1*...*Mn + T1 + ... + Tk depends on column j of Mn and of every Tk only, so device `rank` evaluates
 *     X[:, begin:end] = M1 * ... * M(n-1) * Mn[:, begin:end] + T1[:, begin:end] + ... + Tk[:, begin:end]
 * as an ordinary equation of its own, with no exchange between devices; the slabs of X are the result (gathered
 * by the caller where the whole X is wanted).
 * mom_column_slab: the slab of device `rank`: the `cols` columns are cut into units of `multiple` columns (the last
 * unit may be short) and the units are dealt out contiguously, as evenly as whole units allow; *begin == *end
 * means the device has nothing to do.  multiple = 4 keeps every slab addressable by the tensor-core kernel.
 * Errors: INVALID_ARG (cols < 1, world < 1, rank outside [0, world), multiple < 1, NULL outputs). */
mom_status_t mom_column_slab(int64_t cols, int32_t rank, int32_t world, int64_t multiple, int64_t *begin, int64_t *end);

/* Descriptor of the STORED matrix that holds columns [begin, end) of an operand as used: `stored` describes the
 * whole operand as stored, `transposed` says the equation uses its transpose (then the slab is rows
 * [begin, end) of the stored matrix, contiguous in memory).  The whole operand keeps its property; a proper slab
 * is general (a slab of a triangular, Diagonal, Symmetric or Identity matrix is stored densely with its zeros and
 * ones, the caller's copy).  Errors: those of mom_matrix_desc for `stored`, INVALID_ARG (NULL, begin < 0,
 * end <= begin, end beyond the operand's columns as used). */
mom_status_t mom_column_slab_desc(const mom_matrix_desc_t *stored, int32_t transposed, int64_t begin, int64_t end,
                                  mom_matrix_desc_t *slab);

/* Plan X = prod(chain) + sum(add_terms) (paper Section 2, "Transformations").  Host only: makes no
 * CUDA call and works on a machine without a GPU.
 *   chain      host array of n_chain >= 1 descriptors, left to right
 *   add_terms  host array of n_add >= 0 descriptors (may be NULL when n_add == 0); each must have X's shape
 *   out_plan   receives a plan owned by the caller; release with mom_plan_destroy
 * The multiplication count of a product counts a_il*b_lj only when both factors are structurally
 * non-zero; Identity operands are removed first; among equal-cost parenthesizations the split
 * positions are compared outermost-first, left subtree before right, smallest wins.
 * Errors: INVALID_ARG, PROPERTY, DTYPE, LIMIT, SHAPE_MISMATCH, OVERFLOW, ALLOC.
 * Size limits: a dimension above 2^31 - 1025 is refused (LIMIT); a product with more than 2^24 - 1024 rows or
 * columns never runs on the tcgen05 kernel (its tile table keeps a row index in 24 bits) but on the warp-level
 * or FFMA kernel. */
mom_status_t mom_equation_plan(const mom_matrix_desc_t *chain, int32_t n_chain,
                               const mom_matrix_desc_t *add_terms, int32_t n_add,
                               mom_variant_t variant, mom_plan_t **out_plan);

/* The same with Transpose (paper Table 1, "Transpose"; Section 2 prints the inference rule
 * lowerTriangular(A) -> upperTriangular(A^T)): chain_transposed[i] != 0 means the equation uses the transpose
 * of chain operand i, add_transposed[i] likewise for the Add terms; either array may be NULL (nothing
 * transposed).  The descriptors describe the matrices AS STORED; a transposed operand takes part with its
 * shape swapped and lowerTri <-> upperTri.  Nothing is moved in memory: the kernels read a transposed operand
 * through its stored layout.  In the parenthesization string a transposed operand prints as "i^T". */
mom_status_t mom_equation_plan_transposed(const mom_matrix_desc_t *chain, const int32_t *chain_transposed, int32_t n_chain,
                                          const mom_matrix_desc_t *add_terms, const int32_t *add_transposed, int32_t n_add,
                                          mom_variant_t variant, mom_plan_t **out_plan);

/* Storage of a matrix in device (or host) memory.  The paper materialises every matrix as a dense buffer and names
 * "more appropriate containers" as future work (Section 2, "Matrix Attribute"; the conclusion speaks of
 * non-rectangular iteration spaces).  MOM_STORAGE_PACKED is such a container for triangular matrices (lowerTri,
 * upperTri and their strict and unit kinds): only the triangle is kept, row by row, every stored row a whole number
 * of 16-byte groups so that rows stay addressable by 16-byte accesses:
 *     lower triangle, n x n: row i holds columns [0, 4 * (i / 4 + 1))
 *     upper triangle, n x n: row i holds columns [4 * (i / 4), n rounded up to a multiple of 4)
 * Rows follow each other without gaps.  The stored entries outside the triangle (fewer than four per row, next to
 * the diagonal) and those beyond column n - 1 are padding: zeros in operands (the library relies on it), +0.0f in
 * results.  A packed n x n triangle takes about n (n + 4) / 2 entries instead of n * n. */
typedef enum { MOM_STORAGE_DENSE = 0, MOM_STORAGE_PACKED = 1 } mom_storage_t;

/* Size of the packed container of a rows x rows triangle with the given property, in f32 entries, and where row
 * `row` sits in it: *offset = position of its first stored entry, columns [*first_col, *end_col).
 * Errors: INVALID_ARG (NULL, rows < 1, row outside [0, rows)), PROPERTY (not a triangular property), LIMIT. */
mom_status_t mom_packed_elements(int64_t rows, mom_property_t property, int64_t *elements);
mom_status_t mom_packed_row(int64_t rows, mom_property_t property, int64_t row, int64_t *offset, int64_t *first_col,
                            int64_t *end_col);

/* mom_equation_plan_transposed with a storage per operand, per Add term and for the result.
 *   chain_storage / add_storage   host arrays of mom_storage_t (NULL: all dense); a packed operand must be triangular
 *   result_storage                MOM_STORAGE_PACKED: X is written as a packed triangle; the equation's inferred
 *                                 result type must then be triangular (PROPERTY otherwise)
 * Descriptors still describe the matrices as stored (a packed lower triangle used transposed takes part as an upper
 * one).  The plan is the same as for dense storage (storage changes neither costs nor parenthesization).  Execution:
 * the operand-split pass of the tcgen05 kernel and the batched small-chain kernel read packed operands in place, and
 * the tcgen05 kernel writes a packed X in place (tiles outside the triangle are not written at all); every other
 * kernel gets a dense copy in the workspace (one unpacking pass per packed operand) or leaves a dense X there that a
 * packing pass copies out -- mom_plan_workspace_bytes includes that room.  In mom_equation_execute_batched the
 * instance stride of a packed matrix must be at least its packed size (and a multiple of 4).
 * Errors: those of mom_equation_plan_transposed, PROPERTY (packed storage of a matrix that is not triangular). */
mom_status_t mom_equation_plan_stored(const mom_matrix_desc_t *chain, const int32_t *chain_transposed, const int32_t *chain_storage,
                                      int32_t n_chain, const mom_matrix_desc_t *add_terms, const int32_t *add_transposed,
                                      const int32_t *add_storage, int32_t n_add, mom_storage_t result_storage,
                                      mom_variant_t variant, mom_plan_t **out_plan);

/* Number of f32 entries of X as the plan writes it: rows * cols of the result descriptor, or the packed size. */
mom_status_t mom_plan_result_elements(const mom_plan_t *plan, int64_t *elements);

/* Plan a sum of several Mul chains, X = prod(chain_0) + prod(chain_1) + ... (paper Section 2, "Operations":
 * Mul and Add are both variadic and one Equation holds a bag of them).  A chain of one factor is a plain Add term.
 *   factors            host array with all chains' factors one after the other, AS STORED (n = sum of chain_lengths)
 *   factor_transposed  host array of n flags, or NULL: the equation uses the transpose of that factor
 *   factor_names       host array of n integers, or NULL: factors with equal names are the same stored matrix
 *                      (they must then have equal descriptors, and execute must be given equal pointers and strides
 *                      for them); NULL means that nothing is known to be shared
 *   chain_lengths      host array of n_chains >= 1 lengths, each >= 1
 * Every chain is parenthesized on its own by the rules of mom_equation_plan.  With names, a product below the
 * root of a chain's tree whose run of factors (names and transposition flags) an earlier chain has already
 * multiplied, also below its root, is computed once and read by both; a chain's root product is never shared.
 * Value ids in the steps: 0..n-1 are the factors in the order given, n.. the products in emission order (chain
 * by chain, post-order, shared products once).  The parenthesization string joins the chains' strings with "+".
 * The plan executes through mom_equation_execute / _batched / _host with chain_ptrs holding one pointer per
 * factor (n_add = 0).  All chains must have X's shape.  Errors as mom_equation_plan. */
mom_status_t mom_equation_plan_sum(const mom_matrix_desc_t *factors, const int32_t *factor_transposed,
                                   const int32_t *factor_names, const int32_t *chain_lengths, int32_t n_chains,
                                   mom_variant_t variant, mom_plan_t **out_plan);

/* Nested expressions (paper Section 2, "Operations": the body of an Equation is a bag of Mul, Add and Transpose
 * operations walked from the yield, so they may nest: A*(B + C), (A + B)^T*C, ...).  The expression is a tree
 * (or DAG) of nodes; node `root` is the value X. */
typedef enum {
    MOM_EXPR_OPERAND = 0,    /* operand `operand` of the operand table */
    MOM_EXPR_MUL = 1,        /* product of its children, left to right */
    MOM_EXPR_ADD = 2,        /* sum of its children */
    MOM_EXPR_TRANSPOSE = 3   /* transpose of its single child */
} mom_expr_kind_t;

typedef struct {
    int32_t kind;            /* mom_expr_kind_t */
    int32_t operand;         /* MOM_EXPR_OPERAND: index into `operands`; otherwise ignored */
    int32_t first_child;     /* the node's children are children[first_child .. first_child + n_children), each a */
    int32_t n_children;      /* node index; ignored for MOM_EXPR_OPERAND */
} mom_expr_node_t;

/* Plan an expression.  Host only.
 *   operands   host array of n_operands descriptors, the matrices AS STORED; an operand may be used many times
 *   nodes      host array of n_nodes nodes;  children: host array of n_children node indices;  root: node of X
 * What the planner does with the tree: transposes are pushed down to the operands ((e1*e2)^T = e2^T*e1^T,
 * (e1+e2)^T = e1^T+e2^T); a product inside a product and a sum inside a sum are flattened; a sum inside a
 * product is evaluated on its own, as by mom_equation_plan_sum, into a temporary in the workspace whose type is
 * the sum's result type, and the temporary is one factor of the outer chain (nothing is distributed); nested
 * sums with the same normal form are one temporary.  Products are shared within one sum as described for
 * mom_equation_plan_sum, operands being named by their index.
 * The plan executes through mom_equation_execute / _batched / _host with chain_ptrs holding ONE POINTER PER
 * OPERAND (n_operands entries; an unused or Identity operand may be NULL) and no Add terms.
 * In the parenthesization string an operand prints as its index (with ^T), a temporary as "[" its sum "]".
 * Value ids in the steps count every factor of every chain (nested sums first) and then the products.
 * Errors: INVALID_ARG (bad index, empty operation, a cycle), PROPERTY, DTYPE, SHAPE_MISMATCH, OVERFLOW, ALLOC. */
mom_status_t mom_expression_plan(const mom_matrix_desc_t *operands, int32_t n_operands,
                                 const mom_expr_node_t *nodes, int32_t n_nodes,
                                 const int32_t *children, int32_t n_children, int32_t root,
                                 mom_variant_t variant, mom_plan_t **out_plan);

/* Number of nested sums the plan materializes (0 for plans of the other entry points). */
mom_status_t mom_plan_temporaries(const mom_plan_t *plan, int32_t *temporaries);

/* Number of products that mom_equation_plan_sum did not emit because an earlier chain computes them (0 for
 * plans of the other entry points). */
mom_status_t mom_plan_reused_products(const mom_plan_t *plan, int32_t *reused);

/* mul_flops = 2 * (useful multiplications of the chosen parenthesization; over all chains, a shared product
 * once); add_flops = structural non-zeros of every summand after the first chain: the Add terms (an Identity
 * term counts its n diagonal entries) and the values of the further chains.  Either may be NULL. */
mom_status_t mom_plan_flops(const mom_plan_t *plan, uint64_t *mul_flops, uint64_t *add_flops);

/* The chosen parenthesization over ORIGINAL operand indices, e.g. "(0*(1*3))".  Eliminated Identity
 * operands do not appear; a single surviving operand is its bare index; an all-Identity chain is "I".
 * Writes a NUL-terminated string into buf (host, capacity cap); *needed (optional) receives the
 * size including the NUL.  BUFFER_TOO_SMALL if cap < needed (needed is still written). */
mom_status_t mom_plan_parenthesization(const mom_plan_t *plan, char *buf, size_t cap, size_t *needed);

/* The binary products the variadic Mul was rewritten into (paper Section 2, "Operations": after the symbolic
 * walk the equation is rematerialised as binary multiplications in the optimal order): their number, and
 * product i in execution order (post-order of the tree; 0 <= i < n).  Errors: INVALID_ARG. */
mom_status_t mom_plan_num_steps(const mom_plan_t *plan, int32_t *n);
mom_status_t mom_plan_step(const mom_plan_t *plan, int32_t i, mom_step_t *out);

/* The equation's Term made concrete (paper Section 2, "Types"): shape and inferred property of X. */
mom_status_t mom_plan_result_desc(const mom_plan_t *plan, mom_matrix_desc_t *out);

/* Bytes of device workspace mom_equation_execute[_batched] needs for `batch` instances: room for
 * the intermediates (each also as hi/lo planes for tensor-core steps), the split planes of the
 * operands of tensor-core steps, and split-K partial sums.  May be 0.  (The paper has no counterpart: its
 * bufferization allocates every intermediate with malloc, Section 2, "Matrix Attribute"; here the caller
 * lends one buffer and the plan packs the intermediates into it by live range.)  Errors: INVALID_ARG. */
mom_status_t mom_plan_workspace_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes);

/* Evaluate one equation.
 *   chain_ptrs   host array of n_chain device pointers (entries of Identity operands are ignored)
 *   add_ptrs     host array of n_add device pointers (NULL when n_add == 0)
 *   out          device, rows x cols f32 of the result descriptor
 *   workspace    device, 256-byte aligned, at least mom_plan_workspace_bytes(plan, 1); borrowed for the
 *                duration of the enqueued work; may be NULL when that size is 0
 * The first execution of a plan on a device creates a small plan-owned device block (tile tables,
 * TMA descriptors, a status word) with cudaMalloc; later calls allocate nothing.
 * CUDA graphs: after that first execution the call (and mom_equation_execute_batched) enqueues only kernel
 * launches and, for plans that use their second stream, event records and waits; the caller may capture it on
 * `stream` into a CUDA graph and replay the graph (same bits as the plain call).  The host-staging entry point and
 * mom_product_3xtf32_noalloc are not covered by this statement.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE_TOO_SMALL, ARCH, ALLOC, CUDA. */
mom_status_t mom_equation_execute(const mom_plan_t *plan, const float *const *chain_ptrs,
                                  const float *const *add_ptrs, float *out,
                                  void *workspace, size_t workspace_bytes, mom_stream_t stream);

/* Evaluate `batch` independent instances that share one plan, in one launch sequence.  Instance b of
 * operand i starts at chain_ptrs[i] + b * chain_strides[i] (strides in elements, host arrays;
 * likewise add_strides / out_stride).  Strides must be multiples of 4 elements and at least rows*cols. */
mom_status_t mom_equation_execute_batched(const mom_plan_t *plan, const float *const *chain_ptrs,
                                          const int64_t *chain_strides, const float *const *add_ptrs,
                                          const int64_t *add_strides, float *out, int64_t out_stride,
                                          int64_t batch, void *workspace, size_t workspace_bytes,
                                          mom_stream_t stream);

/* Bytes of device memory mom_equation_execute_host needs as staging: all non-Identity operands, the
 * Add terms, X, and the workspace, for `batch` instances. */
mom_status_t mom_plan_host_staging_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes);

/* Bytes mom_equation_execute_host copies from the host per call: every used operand and Add term once (a
 * named matrix once); of a large triangular operand (batch == 1, at least 1024 rows) only the blocks of 256
 * rows up to (from) the diagonal block are copied, the rest of its device copy is zero-filled on the device. */
mom_status_t mom_plan_host_upload_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes);

/* Same evaluation with HOST operands and a HOST result: copies the operands into `staging` (device,
 * 256-byte aligned, at least mom_plan_host_staging_bytes), runs the plan, copies X back into
 * out_host, all on `stream` (and on two copy streams the plan owns, ordered against `stream` by events: uploads run
 * ahead of the products that need them, a large general operand that an inner tensor-core product reads as its left
 * factor arrives in two pieces and that product starts on the first, and the first rows of a large X travel back
 * while its last rows are still being computed); returns after the stream has been synchronised.  Instances are packed
 * (stride rows*cols).  Pinned host memory makes the copies asynchronous; pageable memory also works. */
mom_status_t mom_equation_execute_host(const mom_plan_t *plan, const float *const *chain_host,
                                       const float *const *add_host, float *out_host, int64_t batch,
                                       void *staging, size_t staging_bytes, mom_stream_t stream);

/* After the stream has been synchronised: code == MOM_OK, or MOM_ERR_DEVICE_TIMEOUT with `detail`
 * identifying the wait that gave up (role << 24 | barrier slot << 16 | low bits of the tile index).
 * Kernels never trap or spin forever: a wait that exceeds its poll limit records this and the CTA
 * leaves cleanly, so the context stays usable.  Reading clears the word. */
mom_status_t mom_plan_device_status(const mom_plan_t *plan, int32_t *code, int32_t *detail);

/* Self-test of the failure route above, without breaking anything: enqueues one tiny kernel in which a single
 * thread waits -- with the very wait routine of the product kernels -- on a barrier that nothing ever signals.
 * After `limit_ms` (0 < limit_ms <= 1000) the wait gives up, records {MOM_ERR_DEVICE_TIMEOUT, detail} in this
 * plan's status block and the kernel ends by itself; once the stream has been synchronised,
 * mom_plan_device_status reports it (and clears it) and the plan executes as before.  (The paper has no
 * counterpart.)  Creates the plan's device state if no execute has done so yet.  Errors: INVALID_ARG, ARCH,
 * ALLOC, CUDA. */
mom_status_t mom_probe_wait_timeout(const mom_plan_t *plan, double limit_ms, int32_t detail, mom_stream_t stream);

/* Steps that run side by side.  Small products leave most of the GPU idle, so where the chosen tree has a product whose two factors
 * are themselves trees of small products (the five-matrix chain ((0*(1*2))*(3*4)): (0*(1*2)) and (3*4)), the launcher runs the right
 * subtree, steps [*begin, *end), on a second stream the plan owns while the left one runs on the caller's stream; step *join waits
 * for both.  (The paper's code generation is sequential; this is the launcher's.)  One such pair per plan; *join = -1: none.  Used for
 * single equations with device operands (not by the batched and host entry points, nor while step timing is on).  The caller sees
 * one stream: everything of an execute is ordered after what the stream held before and before what is enqueued after. */
mom_status_t mom_plan_concurrent_steps(const mom_plan_t *plan, int32_t *begin, int32_t *end, int32_t *join);

/* Number of kernels the most recent execute of this plan enqueued (0 before the first). */
mom_status_t mom_plan_last_launch_count(const mom_plan_t *plan, int32_t *launches);

/* Per-kernel device timing for roofline reports.  With timing enabled every execute brackets each
 * product kernel (and, separately, its operand-split pre-pass) with CUDA events on the caller's stream.
 * After the stream has been synchronised, mom_plan_step_times returns for step i the milliseconds spent
 * in the product kernel and in its pre-pass (0 when there is none), averaged over the executes made since
 * timing was enabled (at most the 32 most recent).
 * Off by default; enabling it creates events but no device memory. */
mom_status_t mom_plan_enable_step_timing(mom_plan_t *plan, int32_t enable);
mom_status_t mom_plan_step_times(const mom_plan_t *plan, int32_t i, float *product_ms, float *prepass_ms);

/* Releases the plan and the launcher state it owns (device block, events, copy streams).  The paper has no
 * counterpart (its plans are compiled code).  NULL is accepted.  Must not run while another thread is inside a
 * call on the same plan.  Kernels of this plan that are still in flight are waited for (the device block is
 * released with cudaFree, which returns once the device has finished with it). */
mom_status_t mom_plan_destroy(mom_plan_t *plan);

const char *mom_status_string(mom_status_t status);

/* One product C = A * B on the tensor-core (3xTF32) kernel without any allocation.  (The paper has no
 * counterpart: this entry point exists for callers of this library, not for the method.)
 *
 * Who needs it: code that may not call cudaMalloc at the point where it needs a product -- for
 * example a plug-in running inside a host application that owns and budgets all device memory, or
 * a latency-critical loop where an allocation (which may synchronise the device) is not acceptable,
 * and that has no spare buffer to lend as workspace.  mom_equation_execute needs a caller workspace
 * and creates a small plan-owned block on first use; this call needs neither.  Its scratch (the hi
 * and lo planes of both operands, the tile table, a status word) is a fixed array of 16 MiB + 33 KiB
 * built into the library; every GPU that loads the library holds that much memory until the process
 * exits.
 *
 *   A (m x k), B (k x n), C (m x n): device, dense row-major f32, 16-byte aligned; k and n multiples of 4.
 *   pa, pb: MOM_GENERAL, MOM_LOWER_TRI or MOM_UPPER_TRI (triangular operands square, zeros stored
 *           outside the triangle); C gets the product's structure (L*L lower, U*U upper, else general)
 *           with +0.0f outside it.
 *   device_status: optional device pointer to 4 ints that the caller has zeroed; receives
 *           {MOM_ERR_DEVICE_TIMEOUT, detail} if a bounded device-side wait expires.  NULL: an internal
 *           word is used (cleared by each call) and the outcome cannot be read back.
 * Limits: 2*(m*k + k*n)*4 bytes (each plane rounded up to 256 bytes) must fit in 16 MiB -- e.g.
 * 1024 x 1024 times 1024 x 1024 -- and the output may have at most 2048 tiles of 128 x 256; beyond that
 * MOM_ERR_LIMIT is returned and nothing is enqueued.  Other errors: INVALID_ARG, PROPERTY, ALIGNMENT,
 * ARCH, CUDA.
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call before any stream capture.  No cudaMalloc, cudaFree or other allocating routine is
 * called.  Asynchronous on `stream`.  All calls on a device share the one array, which keeps the last
 * call's contents (each call rewrites what it reads and clears its status word): two calls that may
 * overlap on the GPU -- different streams without ordering -- race and give wrong results. */
mom_status_t mom_product_3xtf32_noalloc(int64_t m, int64_t n, int64_t k, mom_property_t pa, mom_property_t pb,
                                        const float *A, const float *B, float *C, int32_t *device_status,
                                        mom_stream_t stream);

/* Sustained-rate probes used as roofline denominators.  Each runs an instruction-issue loop on every
 * SM for about `milliseconds` and returns the achieved rate; no global memory traffic besides a
 * few words of output.  `scratch` is device memory of at least 1 MiB.
 *   mom_probe_tf32_tflops:  tcgen05.mma kind::tf32, M=128 N=256 K=8 on resident shared-memory tiles.
 *   mom_probe_ffma_tflops:  independent f32 FMA chains. */
mom_status_t mom_probe_tf32_tflops(double milliseconds, void *scratch, mom_stream_t stream, double *tflops);
mom_status_t mom_probe_ffma_tflops(double milliseconds, void *scratch, mom_stream_t stream, double *tflops);

#ifdef __cplusplus
}
#endif
#endif /* MOM_H_ */
