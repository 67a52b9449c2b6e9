// Host-side Huffman construction for one layer (Sec. IV-A (ii) of arXiv 2204.08211):
// optimal prefix code for the symbol weights, made deterministic and canonical.
//
// Two-queue method: leaves sorted once by (weight, symbol) feed queue A, merged nodes are
// appended to queue B (their weights are non-decreasing), and each step takes the two smallest
// heads, queue A winning ties.  That realises the tie order the interface documents: a leaf before
// a merged node, leaves by symbol, merged nodes by age.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>

#include "co3.h"

namespace {

bool fmt_valid(const co3_fmt& f) {
    if (f.exp_bits < 2 || 1u + f.exp_bits + f.mant_bits > 8u) return false;
    if (f.flags & ~CO3_FMT_FLUSH_SUBNORMALS) return false;
    if (!(f.scale > 0.0f) || !(f.inv_scale > 0.0f)) return false;
    if (std::isinf(f.scale) || std::isinf(f.inv_scale)) return false;
    return true;
}

// A symbol can be produced iff its exponent code is not all ones, it is not "minus zero", and
// (when sub-normal levels are flushed) exponent code 0 carries mantissa code 0.
bool symbol_valid(const co3_fmt& f, unsigned sym) {
    const unsigned nb = f.exp_bits + f.mant_bits;
    if (sym >= (2u << nb)) return false;
    const unsigned sign = sym >> nb, mag = sym & ((1u << nb) - 1u);
    const unsigned efield = mag >> f.mant_bits, mfield = mag & ((1u << f.mant_bits) - 1u);
    if (efield == (1u << f.exp_bits) - 1u) return false;
    if (mag == 0) return sign == 0;
    if (efield == 0 && (f.flags & CO3_FMT_FLUSH_SUBNORMALS) && mfield != 0) return false;
    return true;
}

struct Node {
    uint64_t w;
    int left, right;  // children (node indices) or -1 for a leaf
    int sym;
};

// Depth of every leaf below `root`, iteratively.
void leaf_depths(const Node* nodes, int root, int* depth_of_sym) {
    int stack[1024], dstack[1024], sp = 0;
    stack[sp] = root; dstack[sp] = 0; ++sp;
    while (sp) {
        --sp;
        const int n = stack[sp], d = dstack[sp];
        if (nodes[n].left < 0) { depth_of_sym[nodes[n].sym] = d; continue; }
        stack[sp] = nodes[n].left; dstack[sp] = d + 1; ++sp;
        stack[sp] = nodes[n].right; dstack[sp] = d + 1; ++sp;
    }
}

}  // namespace

extern "C" int co3_code_build(const uint64_t* weights, const co3_fmt* fmt, co3_code* out) {
    if (!weights || !fmt || !out || !fmt_valid(*fmt)) return CO3_ERR_INVALID_ARG;

    int syms[256], n = 0;
    uint64_t w[256];
    uint64_t total = 0;
    for (unsigned s = 0; s < 256; ++s) {
        if (!symbol_valid(*fmt, s)) continue;
        const uint64_t ws = weights[s] ? weights[s] : 1;
        if (ws >= (1ull << 63) || total + ws >= (1ull << 63)) return CO3_ERR_INVALID_ARG;
        total += ws;
        syms[n] = (int)s;
        w[n] = ws;
        ++n;
    }
    std::memset(out, 0, sizeof(*out));
    if (n < 2) return CO3_ERR_INVALID_ARG;

    int len[256];
    for (;;) {
        // queue A: leaves by (weight, symbol); syms[] is already in symbol order, so a stable sort on weight does it
        int order[256];
        for (int i = 0; i < n; ++i) order[i] = i;
        std::stable_sort(order, order + n, [&](int a, int b) { return w[a] < w[b]; });
        Node nodes[512];
        for (int i = 0; i < n; ++i) nodes[i] = Node{w[order[i]], -1, -1, syms[order[i]]};
        int a_head = 0, b_head = n, b_tail = n;
        auto take = [&]() {
            // smaller head; the leaf queue wins ties
            if (a_head < n && (b_head == b_tail || nodes[a_head].w <= nodes[b_head].w)) return a_head++;
            return b_head++;
        };
        for (int k = 0; k < n - 1; ++k) {
            const int x = take();
            const int y = take();
            nodes[b_tail] = Node{nodes[x].w + nodes[y].w, x, y, -1};
            ++b_tail;
        }
        std::memset(len, 0, sizeof(len));
        leaf_depths(nodes, b_tail - 1, len);
        int maxlen = 0;
        for (int i = 0; i < n; ++i) maxlen = std::max(maxlen, len[syms[i]]);
        if (maxlen <= CO3_MAX_CODE_LEN) break;
        for (int i = 0; i < n; ++i) w[i] = std::max<uint64_t>(1, w[i] >> 1);
    }

    // canonical codewords: by (length, symbol), consecutive, shifted when the length grows
    int by_len[256];
    for (int i = 0; i < n; ++i) by_len[i] = syms[i];
    std::stable_sort(by_len, by_len + n, [&](int a, int b) { return len[a] < len[b]; });
    uint32_t code = 0;
    for (int i = 0; i < n; ++i) {
        const int s = by_len[i];
        if (i > 0) code = (code + 1u) << (len[s] - len[by_len[i - 1]]);
        out->len[s] = (uint8_t)len[s];
        out->bits[s] = (uint16_t)code;
    }
    return CO3_OK;
}
