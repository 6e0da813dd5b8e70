"""Table 1 of the paper, executed literally: the per-attribute loops that enumerate the stored
coordinates of a tensor from its pos/crd arrays.

    D : for i from 0 to pos[0]                      -> coordinate i,     position m * pos[0] + i
    CU: for i from pos[m] to pos[m+1]: idx = crd[i] -> coordinate idx,   position i
    CN: for i from pos[0] to pos[1]:  idx = crd[i]  -> coordinate idx,   position i
    S : idx = crd[m]                                -> coordinate idx,   position m

(m is the position produced by the level above, 0 at the first level.) This is an independent reader
of the packed layout: it shares nothing with either packing implementation.
"""


def enumerate_entries(attr, pos, crd):
    """Yield (leaf position, coordinates in storage-level order) for every stored leaf position."""
    order = len(attr)
    out = []

    def walk(level, m, coords):
        if level == order:
            out.append((m, tuple(coords)))
            return
        a = attr[level]
        if a == 0:      # D
            size = int(pos[level][0])
            for i in range(size):
                walk(level + 1, m * size + i, coords + [i])
        elif a == 1:    # CU
            for i in range(int(pos[level][m]), int(pos[level][m + 1])):
                walk(level + 1, i, coords + [int(crd[level][i])])
        elif a == 2:    # CN
            for i in range(int(pos[level][0]), int(pos[level][1])):
                walk(level + 1, i, coords + [int(crd[level][i])])
        else:           # S
            walk(level + 1, m, coords + [int(crd[level][m])])

    walk(0, 0, [])
    return out
