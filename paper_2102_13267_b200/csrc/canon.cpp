// Canonical form of the pending graph and its hash (the compile-cache key, Section 4).
//
// The graph reachable from the roots is linearised in post-order -- roots in creation
// order of the tensors that name them, operands left to right -- so the same program
// traced twice gives the same instruction list whatever tensor ids, arena slots or
// device addresses it used.  Operands are named by canonical index (like %0..%7 in
// Fig. 1), which keeps a*a and a*b apart.  Device-data leaves become parameter ordinals
// by first visit.  Scalars 0 and 1 keep their value in the serialised form; all other
// scalars, and the Philox seed/offset, become numbered run-time slots whose values are
// not serialised (Section 4.1).
#include <cstring>

#include "engine.h"

namespace lt {

namespace {

inline uint64_t rotl(uint64_t x, int r) { return (x << r) | (x >> (64 - r)); }

inline uint64_t avalanche(uint64_t x) {
    x ^= x >> 31;
    x *= 0x7fb5d329728ea185ull;
    x ^= x >> 27;
    x *= 0x81dadef4bc2dd44dull;
    x ^= x >> 33;
    return x;
}

}  // namespace

// 128-bit non-cryptographic hash: two 64-bit lanes, each absorbing every 8-byte word with
// its own rotate-multiply step, cross-mixed and avalanched at the end.
void hash_bytes(const uint8_t *data, size_t n, uint64_t out[2]) {
    uint64_t a = 0x9e3779b97f4a7c15ull ^ (uint64_t)n, b = 0xc2b2ae3d27d4eb4full + (uint64_t)n * 0x165667b19e3779f9ull;
    size_t i = 0;
    for (; i + 8 <= n; i += 8) {
        uint64_t w;
        memcpy(&w, data + i, 8);
        a = rotl(a ^ w, 29) * 0xff51afd7ed558ccdull + 0x52dce729ull;
        b = rotl(b + w * 0x9fb21c651e98df25ull, 37) * 0xc4ceb9fe1a85ec53ull ^ (w >> 17);
    }
    uint64_t tail = 0;
    if (i < n) memcpy(&tail, data + i, n - i);
    a = rotl(a ^ tail, 29) * 0xff51afd7ed558ccdull;
    b = rotl(b + tail * 0x9fb21c651e98df25ull, 37) * 0xc4ceb9fe1a85ec53ull;
    out[0] = avalanche(a + rotl(b, 23));
    out[1] = avalanche(b ^ rotl(a, 41));
}

void canonicalise(lt_ctx *c, const std::vector<uint32_t> &root_tensors, Canonical &cg) {
    cg.nodes.clear();
    cg.outputs.clear();
    cg.donor_param.clear();
    cg.param_node.clear();
    cg.dyn.clear();
    cg.bytes.clear();
    const uint32_t stamp = ++c->stamp;
    std::vector<Node> &N = c->nodes;

    // buffer -> parameter ordinal of the leaf that names it (-2: named by several leaves)
    std::vector<uint32_t> &buf_stamp = c->buf_stamp;
    std::vector<int32_t> &buf_param = c->buf_param;
    if (buf_stamp.size() < c->buffers.size()) {
        buf_stamp.resize(c->buffers.size(), 0);
        buf_param.resize(c->buffers.size(), -1);
    }
    const uint32_t bstamp = stamp;
    std::vector<uint8_t> &param_taken = c->param_taken;
    param_taken.clear();

    struct Frame {
        uint32_t node;
        uint32_t next;
    };
    static thread_local std::vector<Frame> stack;

    auto finish = [&](uint32_t id) {
        Node &n = N[id];
        n.canon = (uint32_t)cg.nodes.size();
        CNode cn;
        cn.op = n.op;
        cn.dtype = n.dtype;
        cn.rank = n.rank;
        cn.n_in = n.n_in;
        for (int i = 0; i < 3; ++i) cn.in[i] = i < n.n_in ? N[n.in[i]].canon : 0;
        for (int i = 0; i < LT_MAX_RANK; ++i) cn.dims[i] = i < n.rank ? n.dims[i] : 0;
        cn.param = -1;
        cn.dyn = -1;
        cn.sval = 0.0;
        cn.attr0 = 0;
        cn.attr1 = 0;
        cn.output = -1;
        cn.arena = id;
        if (n.op == N_DEVICE_DATA) {
            cn.param = (int32_t)cg.param_node.size();
            cg.param_node.push_back(id);
            if (buf_stamp[n.buffer] == bstamp) buf_param[n.buffer] = -2;
            else {
                buf_stamp[n.buffer] = bstamp;
                buf_param[n.buffer] = cn.param;
            }
        } else if (n.op == N_SCALAR) {
            if (n.flags & NF_DYNAMIC) {
                cn.dyn = (int32_t)cg.dyn.size();
                DynValue v;
                v.d = n.sval;
                cg.dyn.push_back(v);
            } else {
                cn.sval = n.sval;
            }
        } else if (n.op == LT_OP_PHILOX_BITS) {
            cn.dyn = (int32_t)cg.dyn.size();
            DynValue v;
            v.i = n.attr[0];
            cg.dyn.push_back(v);
            v.i = n.attr[1];
            cg.dyn.push_back(v);
        } else if (n.op == LT_OP_CONVERT || n.op == LT_OP_IOTA) {
            cn.attr0 = n.attr[0];
        } else if (n.op >= LT_OP_RESHAPE && n.op <= LT_OP_UPDATE_SLICE) {
            cn.attr0 = n.attr[0];
            cn.attr1 = n.attr[1];
        }
        cg.nodes.push_back(cn);
    };

    for (uint32_t slot : root_tensors) {
        const TensorRec &t = c->tensors[slot];
        const uint32_t root = t.node;
        if (N[root].visit != stamp) {
            stack.clear();
            N[root].visit = stamp;
            stack.push_back({root, 0});
            while (!stack.empty()) {
                Frame &f = stack.back();
                Node &n = N[f.node];
                if (f.next < n.n_in) {
                    uint32_t ch = n.in[f.next++];
                    if (N[ch].visit != stamp) {
                        N[ch].visit = stamp;
                        stack.push_back({ch, 0});
                    }
                } else {
                    uint32_t id = f.node;
                    stack.pop_back();
                    finish(id);
                }
            }
        }
        CNode &cn = cg.nodes[N[root].canon];
        if (cn.output < 0) {
            cn.output = (int32_t)cg.outputs.size();
            cg.outputs.push_back(N[root].canon);
            cg.donor_param.push_back(-1);
        }
        // Donation candidate (Section 4.3): the buffer this tensor named before lt_assign, if it is
        // a parameter of this graph that no live tensor names any more.
        if (t.donor != NONE && cg.donor_param[cn.output] < 0 && buf_stamp[t.donor] == bstamp) {
            int32_t p = buf_param[t.donor];
            if (p >= 0) {
                const Node &leaf = N[cg.param_node[p]];
                const Buffer &b = c->buffers[t.donor];
                bool same = leaf.dtype == cn.dtype && leaf.rank == cn.rank;
                for (int i = 0; same && i < cn.rank; ++i) same = leaf.dims[i] == cn.dims[i];
                if (param_taken.size() < cg.param_node.size()) param_taken.resize(cg.param_node.size(), 0);
                if (same && leaf.tensor_refs == 0 && b.refs == 2 && !param_taken[p]) {
                    param_taken[p] = 1;
                    cg.donor_param[cn.output] = p;
                }
            }
        }
    }

    // serialise (into a buffer sized for the worst case, trimmed afterwards)
    std::vector<uint8_t> &b = cg.bytes;
    b.resize(cg.nodes.size() * (4 + 8 * LT_MAX_RANK + 1 + 12 + 4 + 16) + cg.outputs.size() * 8 + 64);
    uint8_t *w = b.data();
    auto put = [&w](auto v) {
        memcpy(w, &v, sizeof(v));
        w += sizeof(v);
    };
    put((uint32_t)0x4c5a5431u);  // format tag
    put((int64_t)c->opt.fusion);
    put((int64_t)c->opt.fast_math);
    put((int64_t)c->opt.horizontal);
    put((int64_t)c->opt.ieee);
    put((uint32_t)cg.nodes.size());
    for (const CNode &n : cg.nodes) {
        put((uint16_t)n.op);
        put((uint8_t)n.dtype);
        put((uint8_t)n.rank);
        for (int i = 0; i < n.rank; ++i) put((int64_t)n.dims[i]);
        if (n.op == N_DEVICE_DATA) {
            put((int32_t)n.param);
        } else if (n.op == N_SCALAR) {
            put((int32_t)n.dyn);
            if (n.dyn < 0) put((double)n.sval);
        } else {
            put((uint8_t)n.n_in);
            for (int i = 0; i < n.n_in; ++i) put((uint32_t)n.in[i]);
            if (n.op == LT_OP_PHILOX_BITS) put((int32_t)n.dyn);
            if (n.op == LT_OP_CONVERT || n.op == LT_OP_IOTA) put((int64_t)n.attr0);
            if (n.op >= LT_OP_RESHAPE && n.op <= LT_OP_UPDATE_SLICE) {
                put((int64_t)n.attr0);
                put((int64_t)n.attr1);
            }
        }
    }
    put((uint32_t)cg.outputs.size());
    for (size_t k = 0; k < cg.outputs.size(); ++k) {
        put((uint32_t)cg.outputs[k]);
        put((int32_t)cg.donor_param[k]);
    }
    b.resize((size_t)(w - b.data()));
}

}  // namespace lt
