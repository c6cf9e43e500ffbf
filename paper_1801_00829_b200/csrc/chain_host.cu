// Host side of the operator chain: validation and translation of the ABI's
// fo_chain into the flat register program the kernels run, plus small host
// utilities shared by the entry points.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <string>

#include "common.cuh"

namespace fo {

namespace {

int arity(int opcode)
{
    if (opcode < FO_OP_ADD) return 1;
    if (opcode == FO_OP_SEL || opcode == FO_OP_FMA) return 3;
    return 2;
}

// Where an ABI operand lives.  Inputs have fixed registers (see common.cuh);
// temporaries are packed behind them, one register per live range.
struct Alloc {
    ChainUse use;
    int n_sides, n_scalars;
    int base;                           // first temporary register
    int8_t reg_tmp[FO_MAX_TMPS];        // current register of temporary k, or -1
    int def_tmp[FO_MAX_TMPS];           // step that defined the current value
    int last_use[FO_MAX_OPS];           // last step reading the value defined at step s
    bool busy[kRegs];
    int high;                           // registers in use (max index + 1)
    uint32_t side_used;
};

enum { kBad = -1 };

// Class and index checks of one operand byte.  Returns 0 if well-formed.
int check_operand(uint8_t o, const Alloc &al, bool has_imm)
{
    const int cls = o >> 6, idx = o & 0x3f;
    switch (cls) {
        case 0: return idx < FO_MAX_TMPS ? 0 : kBad;
        case 1: return (idx < al.n_sides && idx < FO_MAX_SIDES) ? 0 : kBad;
        case 2: return (idx < al.n_scalars && idx < FO_MAX_SCALARS) ? 0 : kBad;
        default:
            if (o == FO_MAIN) return al.use == kUseRow ? kBad : 0;
            if (o == FO_DOT) return al.use == kUseCell ? kBad : 0;
            if (o == FO_IMM) return has_imm ? 0 : kBad;
            return kBad;
    }
}

// Register (or 0x80 | constant slot) of a readable operand; kBad if undefined.
int locate(uint8_t o, Alloc &al, int imm_slot)
{
    const int cls = o >> 6, idx = o & 0x3f;
    switch (cls) {
        case 0: return al.reg_tmp[idx] >= 0 ? al.reg_tmp[idx] : kBad;
        case 1: al.side_used |= 1u << idx; return (al.use == kUseOuter ? 2 : 1) + idx;
        case 2: return 0x80 | idx;
        default:
            if (o == FO_MAIN) return 0;
            if (o == FO_DOT) return al.use == kUseOuter ? 1 : 0;
            return 0x80 | imm_slot;
    }
}

}  // namespace

int translate_chain(const fo_chain *chain, ChainUse use, int n_sides,
                    const double *scalars, int n_scalars, int min_out, int max_out,
                    DevChain *out)
{
    if (!chain || !out) return FO_ERR_NULL;
    if (chain->n_ops < 0 || chain->n_ops > FO_MAX_OPS) return FO_ERR_CHAIN;
    if (chain->n_ops > 0 && !chain->ops) return FO_ERR_NULL;
    if (chain->n_out < min_out || chain->n_out > max_out || chain->n_out > FO_MAX_OUT)
        return FO_ERR_CHAIN;
    if (n_sides < 0 || n_sides > FO_MAX_SIDES) return FO_ERR_UNSUPPORTED;
    if (n_scalars < 0 || n_scalars > FO_MAX_SCALARS) return FO_ERR_UNSUPPORTED;
    if (n_scalars > 0 && !scalars) return FO_ERR_NULL;
    if (use == kUseOuter && n_sides > kOuterMaxSides) return FO_ERR_UNSUPPORTED;

    memset(out, 0, sizeof(*out));
    Alloc al;
    memset(&al, 0, sizeof(al));
    al.use = use;
    al.n_sides = n_sides;
    al.n_scalars = n_scalars;
    al.base = (use == kUseOuter) ? 2 + n_sides : 1 + n_sides;
    al.high = al.base;
    for (int k = 0; k < FO_MAX_TMPS; ++k) { al.reg_tmp[k] = -1; al.def_tmp[k] = -1; }

    // Pass 1: well-formedness, use-before-definition, last use of every definition.
    const int n = chain->n_ops;
    for (int s = 0; s < n; ++s) {
        const fo_op *op = &chain->ops[s];
        if (op->opcode >= FO_OP_COUNT_ || op->dst >= FO_MAX_TMPS) return FO_ERR_CHAIN;
        const uint8_t src[3] = {op->a, op->b, op->c};
        for (int k = 0; k < arity(op->opcode); ++k) {
            if (check_operand(src[k], al, true) != 0) return FO_ERR_CHAIN;
            if ((src[k] >> 6) == 0) {
                const int d = al.def_tmp[src[k] & 0x3f];
                if (d < 0) return FO_ERR_CHAIN;
                al.last_use[d] = s;
            }
        }
        al.def_tmp[op->dst] = s;
        al.last_use[s] = s;                    // a value nobody reads dies at once
    }
    for (int k = 0; k < chain->n_out; ++k) {
        const uint8_t o = chain->out[k];
        if (check_operand(o, al, false) != 0) return FO_ERR_CHAIN;
        if ((o >> 6) == 0) {
            const int d = al.def_tmp[o & 0x3f];
            if (d < 0) return FO_ERR_CHAIN;
            al.last_use[d] = n;                // results stay live to the end
        }
    }

    // Pass 2: assign registers, freeing a temporary's register after its last read.
    for (int k = 0; k < FO_MAX_TMPS; ++k) al.def_tmp[k] = -1;
    for (int k = 0; k < n_scalars; ++k) out->consts[k] = scalars[k];
    for (int s = 0; s < n; ++s) {
        const fo_op *op = &chain->ops[s];
        const int imm_slot = FO_MAX_SCALARS + s;
        out->consts[imm_slot] = op->imm;
        const uint8_t src[3] = {op->a, op->b, op->c};
        int x[3] = {0, 0, 0};
        for (int k = 0; k < arity(op->opcode); ++k) {
            x[k] = locate(src[k], al, imm_slot);
            if (x[k] == kBad) return FO_ERR_CHAIN;
        }
        // operands are fetched before the result is written, so a register whose
        // value is read here for the last time may receive the result
        for (int k = 0; k < FO_MAX_TMPS; ++k) {
            if (al.reg_tmp[k] >= 0 && al.last_use[al.def_tmp[k]] <= s) {
                al.busy[al.reg_tmp[k]] = false;
                al.reg_tmp[k] = -1;
            }
        }
        if (al.reg_tmp[op->dst] >= 0) {        // overwritten while still marked live
            al.busy[al.reg_tmp[op->dst]] = false;
            al.reg_tmp[op->dst] = -1;
        }
        int r = al.base;
        while (r < kRegs && al.busy[r]) ++r;
        if (r >= kRegs) return FO_ERR_CHAIN;
        al.busy[r] = true;
        al.reg_tmp[op->dst] = (int8_t)r;
        al.def_tmp[op->dst] = s;
        if (r + 1 > al.high) al.high = r + 1;
        DevOp &o = out->ops[s];
        o.opcode = op->opcode;
        o.dst = (uint8_t)r;
        o.a = (uint8_t)x[0];
        o.b = (uint8_t)x[1];
        o.c = (uint8_t)x[2];
    }
    for (int k = 0; k < chain->n_out; ++k) {
        const int x = locate(chain->out[k], al, 0);
        if (x == kBad) return FO_ERR_CHAIN;
        out->out[k] = (uint8_t)x;
    }
    out->n_ops = n;
    out->n_out = chain->n_out;
    out->n_regs = al.high;
    out->side_used = al.side_used;
    out->tmp_base = al.base;
    return FO_OK;
}

int chain_expression(const DevChain &ch, int k, char *text, size_t cap)
{
    static const char *const names[FO_OP_COUNT_] = {
        "mov", "neg", "abs", "sqrt", "exp", "log", "sq", "add", "sub", "mul", "div",
        "min", "max", "pow", "eq", "ne", "lt", "le", "gt", "ge", "sel", "fma"};
    std::string reg[kRegs + 1];
    for (int r = 0; r < kRegs + 1; ++r) reg[r] = "r" + std::to_string(r);
    auto operand_text = [&](int o) -> std::string {
        if (o & 0x80) return "k" + std::to_string(o & 0x7f);
        return (o >= 0 && o <= kRegs) ? reg[o] : std::string("?");
    };
    const size_t limit = 4096;       // shared subexpressions are written out again: bound the growth
    for (int s = 0; s < ch.n_ops; ++s) {
        const DevOp &op = ch.ops[s];
        if (op.opcode >= FO_OP_COUNT_ || op.dst > kRegs) return -1;
        const std::string a = operand_text(op.a);
        std::string e;
        if (op.opcode == FO_OP_MOV) e = a;
        else if (op.opcode == FO_OP_SQ) e = "mul(" + a + "," + a + ")";
        else if (op.opcode < FO_OP_ADD) e = std::string(names[op.opcode]) + "(" + a + ")";
        else if (op.opcode == FO_OP_SEL || op.opcode == FO_OP_FMA)
            e = std::string(names[op.opcode]) + "(" + a + "," + operand_text(op.b) + "," + operand_text(op.c) + ")";
        else e = std::string(names[op.opcode]) + "(" + a + "," + operand_text(op.b) + ")";
        if (e.size() > limit) return -1;
        reg[op.dst] = e;
    }
    if (k < 0 || k >= ch.n_out) return -1;
    const std::string out = operand_text(ch.out[k]);
    if (out.size() + 1 > cap) return -1;
    memcpy(text, out.c_str(), out.size() + 1);
    return 0;
}

int check_workspace(const void *ws, size_t ws_bytes, size_t need)
{
    if (!ws) return FO_ERR_WORKSPACE;
    if (((uintptr_t)ws & 255u) != 0) return FO_ERR_WORKSPACE;
    if (ws_bytes < need) return FO_ERR_WORKSPACE;
    return FO_OK;
}

static thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return FO_ERR_CUDA;
}

int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

// ---- measurement knobs (fo_tune): a small table of named strings.  Kernels read
// a knob at launch; a knob that was never set costs one relaxed atomic load.
namespace {
struct Knob {
    const char *name;
    char value[48];
    bool set;
};
Knob g_knobs[] = {
    {"cell.ctas_per_sm", "", false}, {"row.narrow", "", false},
    {"b1.shape", "", false},         {"b1.mma_shape", "", false},    {"b1.narrow", "", false},
    {"b1.mma", "", false},           {"outer.kernel", "", false},
    {"cell.stamps", "", false},
};
std::mutex g_knob_mutex;
std::atomic<int> g_knobs_set{0};
}  // namespace

bool tune_get(const char *name, char *value, size_t cap)
{
    if (g_knobs_set.load(std::memory_order_relaxed) == 0) return false;
    std::lock_guard<std::mutex> lock(g_knob_mutex);
    for (Knob &k : g_knobs)
        if (k.set && strcmp(k.name, name) == 0) {
            snprintf(value, cap, "%s", k.value);
            return true;
        }
    return false;
}

int tune_int(const char *name, int fallback)
{
    char v[48];
    if (!tune_get(name, v, sizeof(v))) return fallback;
    char *end = nullptr;
    const long x = strtol(v, &end, 10);
    return end != v ? (int)x : fallback;
}

}  // namespace fo

extern "C" {

int fo_tune(const char *name, const char *value)
{
    if (!name) return FO_ERR_NULL;
    std::lock_guard<std::mutex> lock(fo::g_knob_mutex);
    for (fo::Knob &k : fo::g_knobs)
        if (strcmp(k.name, name) == 0) {
            if (value && strlen(value) >= sizeof(k.value)) return FO_ERR_SHAPE;
            const bool was = k.set;
            k.set = value != nullptr;
            if (value) snprintf(k.value, sizeof(k.value), "%s", value);
            fo::g_knobs_set.fetch_add((k.set ? 1 : 0) - (was ? 1 : 0));
            return FO_OK;
        }
    return FO_ERR_UNSUPPORTED;
}

const char *fo_status_string(int status)
{
    switch (status) {
        case FO_OK: return "ok";
        case FO_ERR_NULL: return "a required pointer is NULL";
        case FO_ERR_SHAPE: return "input dimensions do not fit together";
        case FO_ERR_CHAIN: return "invalid operator chain";
        case FO_ERR_UNSUPPORTED: return "variant or size not supported";
        case FO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FO_ERR_CUDA: return "CUDA runtime error at launch";
        case FO_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case FO_ERR_STATIC_LIMIT: return "the call needs more scratch than the built-in array holds";
        default: return "unknown status";
    }
}

int fo_last_cuda_error(void) { return fo::g_last_cuda_error; }

int fo_workspace_init(void *ws, size_t ws_bytes, void *stream)
{
    const int rc = fo::check_workspace(ws, ws_bytes, sizeof(fo::WsHead));
    if (rc != FO_OK) return rc;
    const cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(fo::WsHead), (cudaStream_t)stream);
    return e == cudaSuccess ? FO_OK : fo::cuda_fail(e);
}

int fo_query_device_status(const void *ws, void *stream, int *status)
{
    if (!ws || !status) return FO_ERR_NULL;
    unsigned int words[2] = {0u, 0u};      // ticket, status
    cudaError_t e = cudaMemcpyAsync(words, ws, sizeof(words), cudaMemcpyDeviceToHost,
                                    (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return fo::cuda_fail(e);
    *status = words[1] ? FO_ERR_DEVICE_TIMEOUT : FO_OK;
    return FO_OK;
}

int fo_chain_describe(const fo_chain *chain, int use, int n_sides, const double *scalars, int n_scalars,
                      int k, char *text, size_t cap)
{
    if (!chain || !text || cap == 0) return FO_ERR_NULL;
    if (use < 0 || use > 2) return FO_ERR_SHAPE;
    fo::DevChain ch;
    const int rc = fo::translate_chain(chain, (fo::ChainUse)use, n_sides, scalars, n_scalars, 1, FO_MAX_OUT, &ch);
    if (rc != FO_OK) return rc;
    if (k < 0 || k >= ch.n_out) return FO_ERR_SHAPE;
    return fo::chain_expression(ch, k, text, cap) == 0 ? FO_OK : FO_ERR_SHAPE;
}

}  // extern "C"
