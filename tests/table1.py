"""An independent reader of the packed layout: a walk over (pos, crd) by the level rules of the storage format
(Table 1 of the paper gives them as one loop form per attribute; include/comet.h states them in words):

    D   every coordinate 0 .. pos[0]-1 under each parent position m; the child's position is m * pos[0] + coordinate
    CU  the children of parent position m are the positions pos[m] .. pos[m+1]-1; coordinate crd[position]
    CN  (first level) the positions pos[0] .. pos[1]-1; coordinate crd[position]
    S   one child per parent position m, at the same position; coordinate crd[m]

(m is the position produced by the level above, 0 at the first level.) It shares nothing with either packing
implementation.
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
