"""Tile-span recursions of the paper, written out -- TEST INFRASTRUCTURE ONLY.

A span is an inclusive 1-D interval (a1, a2) of one map axis; the paper writes
the 2-D span of tile (i, j) at map l as top-left (x1, y1), bottom-right
(x2, y2) (Section 4.2).  Both axes follow the same recursion, so everything
here is 1-D and the callers apply it to x and y separately.

Layers are objects with attributes kind ("conv"/"pool"), k, stride, pad.
"""


def eq1_conv(a1, a2, K, S):
    """Eq. (1a-d): span at the input of a conv layer (kernel K, stride S) that
    the output span (a1, a2) depends on, before clamping to the map."""
    return a1 * S - K // 2, a2 * S + K // 2 + (S - 1)


def eq2_conv(a1, a2, K, S):
    """Eq. (2a-d): delta-map span at the output of a conv layer (kernel K,
    stride S) reached from the delta span (a1, a2) at its input.  Uses exact
    integer ceil/floor division."""
    lo = -((-(a1 - K // 2)) // S)       # ceil((a1 - floor(K/2)) / S)
    hi = (a2 + K // 2) // S             # floor((a2 + floor(K/2)) / S)
    return lo, hi


def receptive(a1, a2, K, S, P):
    """General receptive field with explicit padding P: the inputs that the
    outputs a1..a2 of a window op (kernel K, stride S, padding P) read.
    Equals Eq. (1) for odd K, S = 1, P = floor(K/2); gives 2*a1 .. 2*a2+1 for
    the unpadded 2x2/2 pool, for which the paper prints no formula."""
    return a1 * S - P, a2 * S - P + K - 1


def equal_partition(extent, parts):
    """'Partitioned ... equally among the tiles' (Section 4.2): tile i of
    `parts` owns [floor(i*extent/parts), floor((i+1)*extent/parts) - 1]."""
    return [((i * extent) // parts, ((i + 1) * extent) // parts - 1)
            for i in range(parts)]


def clamp(a1, a2, extent):
    return max(a1, 0), min(a2, extent - 1)


def forward_spans(layers, out_extent, out_span):
    """Spans of one tile at every map of a group, from the group's output map
    back to its input map.  `layers` are the group's layers in forward order,
    `out_extent` the extent of the group's output map along this axis.
    Each span is clamped to its map before the recursion continues.
    Returns a list of len(layers)+1 spans, index 0 = group input map."""
    extents = [out_extent]
    for l in reversed(layers):
        extents.append(extents[-1] * l.stride if l.kind == "pool" else extents[-1])
    extents.reverse()
    spans = [None] * (len(layers) + 1)
    spans[-1] = out_span
    for i in range(len(layers) - 1, -1, -1):
        l = layers[i]
        a1, a2 = receptive(spans[i + 1][0], spans[i + 1][1], l.k, l.stride, l.pad)
        spans[i] = clamp(a1, a2, extents[i])
    return spans


def brute_force_dependency(layers, in_extent, out_span):
    """Pin for the recursion: mark, by walking every window of every layer,
    which positions of each map the outputs in `out_span` depend on.  Returns
    per map the (min, max) marked position (positions outside a map are
    padding and are not marked).  Index 0 = group input map."""
    extents = [in_extent]
    for l in layers:
        extents.append((extents[-1] + 2 * l.pad - l.k) // l.stride + 1)
    need = [set() for _ in range(len(layers) + 1)]
    need[-1] = set(range(out_span[0], out_span[1] + 1))
    for i in range(len(layers) - 1, -1, -1):
        l = layers[i]
        for o in need[i + 1]:
            for t in range(l.k):
                p = o * l.stride - l.pad + t
                if 0 <= p < extents[i]:
                    need[i].add(p)
    return [(min(s), max(s)) for s in need]
