// Host-only parts of librtoss: status text, pattern-table presets and
// validation (Section IV.B of arXiv 2303.02191), layer grouping by depth-first
// search (Section IV.A, Algorithm 1).  Plain C++, no CUDA.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <vector>

#include "rtoss.h"
#include "rtoss_internal.h"

namespace {

// neighbours[t] = mask of the taps sharing an edge with tap t in the 3x3 grid
constexpr uint16_t kNeighbours[9] = {
    0x00A, 0x015, 0x022,  // 0:{1,3} 1:{0,2,4} 2:{1,5}
    0x051, 0x0AA, 0x114,  // 3:{0,4,6} 4:{1,3,5,7} 5:{2,4,8}
    0x088, 0x150, 0x0A0   // 6:{3,7} 7:{4,6,8} 8:{5,7}
};

bool edge_connected(unsigned m) {
    unsigned reach = m & (0u - m);
    unsigned frontier = reach;
    while (frontier) {
        unsigned next = 0;
        for (unsigned f = frontier; f; f &= f - 1) next |= kNeighbours[__builtin_ctz(f)];
        next &= m & ~reach;
        reach |= next;
        frontier = next;
    }
    return reach == m;
}

bool is_centre8(unsigned m) {
    // 2x2 blocks through the centre, and the centre with three of its edge neighbours
    static const uint16_t members[8] = {
        (1 << 0) | (1 << 1) | (1 << 3) | (1 << 4), (1 << 1) | (1 << 2) | (1 << 4) | (1 << 5),
        (1 << 3) | (1 << 4) | (1 << 6) | (1 << 7), (1 << 4) | (1 << 5) | (1 << 7) | (1 << 8),
        (1 << 4) | (1 << 1) | (1 << 3) | (1 << 5), (1 << 4) | (1 << 1) | (1 << 3) | (1 << 7),
        (1 << 4) | (1 << 1) | (1 << 5) | (1 << 7), (1 << 4) | (1 << 3) | (1 << 5) | (1 << 7)};
    for (uint16_t x : members)
        if (x == m) return true;
    return false;
}

}  // namespace

bool rtoss_table_ok(const uint16_t* masks, int P, int k) {
    if (!masks || P < 1 || P > 255 || k < 1 || k > 9) return false;
    bool seen[512] = {false};
    for (int p = 0; p < P; ++p) {
        unsigned m = masks[p];
        if (m == 0 || m > 511 || __builtin_popcount(m) != k || seen[m]) return false;
        seen[m] = true;
    }
    return true;
}

extern "C" {

const char* rtoss_status_string(rtoss_status s) {
    switch (s) {
        case RTOSS_OK: return "ok";
        case RTOSS_ERR_INVALID_ARG: return "invalid argument";
        case RTOSS_ERR_BAD_PATTERN_TABLE: return "bad pattern table";
        case RTOSS_ERR_UNSUPPORTED: return "unsupported configuration";
        case RTOSS_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case RTOSS_ERR_ALLOC: return "allocation failed";
        case RTOSS_ERR_CUDA: return "CUDA error";
        case RTOSS_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

rtoss_status rtoss_pattern_preset(int k, rtoss_preset preset, uint16_t* masks_host, int* P) {
    if (!masks_host || !P || *P < 0) return RTOSS_ERR_INVALID_ARG;
    const int cap = *P;
    int n = 0;
    if (preset == RTOSS_PRESET_DENSE) {
        if (k != 9 || cap < 1) return RTOSS_ERR_INVALID_ARG;
        masks_host[0] = 0x1FF;
        *P = 1;
        return RTOSS_OK;
    }
    if (k < 1 || k > 9) return RTOSS_ERR_INVALID_ARG;
    if (preset == RTOSS_PRESET_CENTRE8 && k != 4) return RTOSS_ERR_INVALID_ARG;
    if (preset != RTOSS_PRESET_ALL && preset != RTOSS_PRESET_CONN4 && preset != RTOSS_PRESET_CENTRE8)
        return RTOSS_ERR_INVALID_ARG;
    for (unsigned m = 1; m <= 511; ++m) {
        if (__builtin_popcount(m) != k) continue;
        bool take = preset == RTOSS_PRESET_ALL || (preset == RTOSS_PRESET_CONN4 && edge_connected(m)) ||
                    (preset == RTOSS_PRESET_CENTRE8 && is_centre8(m));
        if (!take) continue;
        if (n == cap) return RTOSS_ERR_INVALID_ARG;
        masks_host[n++] = static_cast<uint16_t>(m);
    }
    *P = n;
    return RTOSS_OK;
}

rtoss_status rtoss_pattern_table_validate(const uint16_t* masks_host, int P, int k) {
    return rtoss_table_ok(masks_host, P, k) ? RTOSS_OK : RTOSS_ERR_BAD_PATTERN_TABLE;
}

rtoss_status rtoss_pattern_rank(const uint16_t* masks_host, const uint64_t* counts_host, int P, int k, int M,
                                uint16_t* top_masks_host, int* order_host) {
    if (!masks_host || !counts_host || !top_masks_host) return RTOSS_ERR_INVALID_ARG;
    if (!rtoss_table_ok(masks_host, P, k)) return RTOSS_ERR_BAD_PATTERN_TABLE;
    if (M < 1 || M > P) return RTOSS_ERR_INVALID_ARG;
    std::vector<int> order(P);
    for (int i = 0; i < P; ++i) order[i] = i;
    std::sort(order.begin(), order.end(), [&](int a, int b) {
        if (counts_host[a] != counts_host[b]) return counts_host[a] > counts_host[b];
        return masks_host[a] < masks_host[b];
    });
    if (order_host)
        for (int i = 0; i < P; ++i) order_host[i] = order[i];
    std::vector<uint16_t> top(M);
    for (int i = 0; i < M; ++i) top[i] = masks_host[order[i]];
    std::sort(top.begin(), top.end());
    for (int i = 0; i < M; ++i) top_masks_host[i] = top[i];
    return RTOSS_OK;
}

rtoss_status rtoss_group_layers(const rtoss_layer_node* nodes, int L, int* parent, int* group, int* n_groups) {
    if (!nodes || !parent || !group || L < 0) return RTOSS_ERR_INVALID_ARG;
    for (int i = 0; i < L; ++i) {
        if (nodes[i].n_inputs < 0 || (nodes[i].n_inputs > 0 && !nodes[i].inputs)) return RTOSS_ERR_INVALID_ARG;
        for (int e = 0; e < nodes[i].n_inputs; ++e)
            if (nodes[i].inputs[e] < 0 || nodes[i].inputs[e] >= i) return RTOSS_ERR_INVALID_ARG;
        if (nodes[i].is_conv && (nodes[i].cout < 1 || nodes[i].cin < 1 || (nodes[i].ksize != 1 && nodes[i].ksize != 3)))
            return RTOSS_ERR_INVALID_ARG;
    }
    // nearest[i]: the first convolution a depth-first walk meets going upstream from node i's
    // inputs (listed order, passing through non-convolution nodes).  Because nodes are in
    // topological order, the answer for a non-convolution input is already known: memoised DFS.
    std::vector<int> nearest(L, -1);
    int groups = 0;
    for (int i = 0; i < L; ++i) {
        int found = -1;
        for (int e = 0; e < nodes[i].n_inputs && found < 0; ++e) {
            int u = nodes[i].inputs[e];
            found = nodes[u].is_conv ? u : nearest[u];
        }
        nearest[i] = found;
        if (!nodes[i].is_conv) {
            parent[i] = -1;
            group[i] = -1;
            continue;
        }
        if (found < 0) {
            parent[i] = i;
            group[i] = groups++;
        } else {
            parent[i] = found;
            const rtoss_layer_node &a = nodes[i], &b = nodes[found];
            group[i] = (a.ksize == b.ksize && a.cout == b.cout && a.cin == b.cin) ? group[found] : groups++;
        }
    }
    if (n_groups) *n_groups = groups;
    return RTOSS_OK;
}

}  // extern "C"
