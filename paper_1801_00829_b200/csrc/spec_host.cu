// Host side of chain specialisation: recognises a translated Cell / MAgg chain
// as one of the compile-time specialisations of spec.cuh.
#include "common.cuh"
#include "spec.cuh"

namespace fo {

namespace {

struct RefOp {
    uint8_t opcode, dst, a, b;
};
struct RefChain {
    int id;
    int n_ops;
    RefOp ops[3];
    int n_out;
    uint8_t out[3];
};

// Reference programs in ABI operand bytes (fusedops.h).
const RefChain kRefs[] = {
    {kSpecMul2, 1, {{FO_OP_MUL, 0, FO_MAIN, FO_SIDE(0)}}, 1, {FO_TMP(0)}},
    {kSpecMul3, 2, {{FO_OP_MUL, 0, FO_MAIN, FO_SIDE(0)}, {FO_OP_MUL, 1, FO_TMP(0), FO_SIDE(1)}}, 1,
     {FO_TMP(1)}},
    {kSpecSq, 1, {{FO_OP_MUL, 0, FO_MAIN, FO_MAIN}}, 1, {FO_TMP(0)}},
    {kSpecSq, 1, {{FO_OP_SQ, 0, FO_MAIN, 0}}, 1, {FO_TMP(0)}},
    {kSpecMagg2, 2, {{FO_OP_MUL, 0, FO_MAIN, FO_SIDE(0)}, {FO_OP_MUL, 1, FO_MAIN, FO_SIDE(1)}}, 2,
     {FO_TMP(0), FO_TMP(1)}},
    {kSpecMagg3, 3,
     {{FO_OP_MUL, 0, FO_MAIN, FO_SIDE(0)}, {FO_OP_MUL, 1, FO_MAIN, FO_SIDE(1)},
      {FO_OP_MUL, 2, FO_MAIN, FO_MAIN}},
     3, {FO_TMP(0), FO_TMP(1), FO_TMP(2)}},
};

// Operand of a translated chain in a form that does not depend on how many
// sides the caller passed: inputs keep their number, temporaries count from 0.
int normal(int opnd, int tmp_base)
{
    if (opnd & 0x80) return -1;                  // constants: no specialisation uses one
    return opnd < tmp_base ? opnd : 100 + (opnd - tmp_base);
}

bool same_program(const DevChain &a, const DevChain &b)
{
    if (a.n_ops != b.n_ops || a.n_out != b.n_out || a.side_used != b.side_used) return false;
    for (int s = 0; s < a.n_ops; ++s) {
        const DevOp &x = a.ops[s], &y = b.ops[s];
        if (x.opcode != y.opcode) return false;
        if (normal(x.dst, a.tmp_base) != normal(y.dst, b.tmp_base)) return false;
        const int na = normal(x.a, a.tmp_base), nb = normal(y.a, b.tmp_base);
        if (na < 0 || na != nb) return false;
        if (x.opcode >= FO_OP_ADD) {
            const int ma = normal(x.b, a.tmp_base), mb = normal(y.b, b.tmp_base);
            if (ma < 0 || ma != mb) return false;
        }
        if (x.opcode == FO_OP_SEL || x.opcode == FO_OP_FMA) return false;
    }
    for (int k = 0; k < a.n_out; ++k) {
        const int na = normal(a.out[k], a.tmp_base), nb = normal(b.out[k], b.tmp_base);
        if (na < 0 || na != nb) return false;
    }
    return true;
}

// side0 + (a * c) * side1 with c a scalar or an immediate, in either operand order of
// each step (multiplication and addition commute bit for bit).  Returns the constant's
// slot, or -1.  Inputs: register 0 = a, 1 = side 0, 2 = side 1.
int scaled_add_slot(const DevChain &ch)
{
    if (ch.n_ops != 3 || ch.n_out != 1 || ch.side_used != 3u) return -1;
    const DevOp &m0 = ch.ops[0], &m1 = ch.ops[1], &ad = ch.ops[2];
    if (m0.opcode != FO_OP_MUL || m1.opcode != FO_OP_MUL || ad.opcode != FO_OP_ADD) return -1;
    int slot = -1;
    if (m0.a == 0 && (m0.b & 0x80)) slot = m0.b & 0x7f;
    else if (m0.b == 0 && (m0.a & 0x80)) slot = m0.a & 0x7f;
    if (slot < 0 || m0.dst < ch.tmp_base) return -1;
    if (!((m1.a == m0.dst && m1.b == 2) || (m1.b == m0.dst && m1.a == 2))) return -1;
    if (!((ad.a == 1 && ad.b == m1.dst) || (ad.b == 1 && ad.a == m1.dst))) return -1;
    if (ch.out[0] != ad.dst) return -1;
    return slot;
}

}  // namespace

int scaled_add_const(const DevChain &ch) { return scaled_add_slot(ch); }

int match_cell_spec(const DevChain &ch)
{
    if (scaled_add_slot(ch) >= 0) return kSpecScaledAdd;
    for (const RefChain &r : kRefs) {
        fo_op ops[3];
        memset(ops, 0, sizeof(ops));
        for (int s = 0; s < r.n_ops; ++s) {
            ops[s].opcode = r.ops[s].opcode;
            ops[s].dst = r.ops[s].dst;
            ops[s].a = r.ops[s].a;
            ops[s].b = r.ops[s].b;
        }
        fo_chain c;
        memset(&c, 0, sizeof(c));
        c.n_ops = r.n_ops;
        c.n_out = r.n_out;
        c.ops = ops;
        for (int k = 0; k < r.n_out; ++k) c.out[k] = r.out[k];
        DevChain ref;
        if (translate_chain(&c, kUseCell, 2, nullptr, 0, 1, FO_MAX_OUT, &ref) != FO_OK) continue;
        // a * a written with the square opcode is the same arithmetic as mul(a, a)
        if (r.id == kSpecSq && r.ops[0].opcode == FO_OP_SQ) {
            if (ch.n_ops == 1 && ch.n_out == 1 && ch.ops[0].opcode == FO_OP_SQ && ch.ops[0].a == 0 &&
                ch.out[0] == ch.ops[0].dst && ch.side_used == 0)
                return kSpecSq;
            continue;
        }
        if (same_program(ch, ref)) return r.id;
    }
    return kSpecNone;
}

}  // namespace fo
