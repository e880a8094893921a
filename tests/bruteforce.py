"""Brute-force model of one pruning step for tiny inputs: pure Python loops, numpy
float32 scalars, and a FULL sort of every layer by (importance descending, index
ascending).  It exists to pin the oracle (which uses a library partial-ordering
routine) and is far too slow for anything but a few hundred elements."""
import math

import numpy as np

F = np.float32


def bits(x) -> int:
    return int(np.asarray(x, dtype=np.float32).view(np.uint32))


def importance(a, w, eps):
    return F(abs(F(a))) / (F(abs(F(w))) + F(eps))


class BruteForce:
    def __init__(self, layer_sizes, W, ratio, eps, momentum=1.0):
        self.m = F(momentum)
        self.n = list(layer_sizes)
        self.W, self.ratio, self.eps = W, float(ratio), F(eps)
        self.N = sum(self.n)
        self.k = [min(n, max(1, math.ceil(n / self.ratio))) for n in self.n]
        self.acc = [[F(0)] * self.N for _ in range(W)]

    def step(self, grads, weights, leader):
        W, N = self.W, self.N
        for w in range(W):
            for i in range(N):
                self.acc[w][i] = F(F(self.m * self.acc[w][i]) + F(grads[w][i]))
        lists = []
        for w in range(W):
            lst, o = [], 0
            for n, k in zip(self.n, self.k):
                imp = [bits(importance(self.acc[w][o + i], weights[o + i], self.eps)) for i in range(n)]
                ranked = sorted(range(n), key=lambda i: (-imp[i], i))
                lst += [(o + i, self.acc[w][o + i]) for i in sorted(ranked[:k])]
                o += n
            lists.append(lst)
        S = [i for i, _ in lists[leader]]
        update = [F(0)] * N
        for i in S:
            s = self.acc[0][i]
            for w in range(1, W):
                s = F(s + self.acc[w][i])
            update[i] = F(F(0) + s)
        for i in S:
            for w in range(W):
                self.acc[w][i] = F(0)
        return lists, np.array(update, dtype=np.float32)

    def residual(self, w):
        return np.array(self.acc[w], dtype=np.float32)
