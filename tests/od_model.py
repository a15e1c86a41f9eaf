"""A second, independent statement of the cache table on Python's OrderedDict — the container type the
paper's prototype uses (Section 3.1).  Recency is the dict order itself (move_to_end / popitem), with no
clock, so it shares no mechanism with the oracle's stamp counters."""
from collections import OrderedDict


class ODTable:
    def __init__(self, LL, FL, LC, FC, refresh_on_reinsert=True):
        self.LL, self.FL, self.LC, self.FC = LL, FL, LC, FC
        self.refresh = refresh_on_reinsert
        self.t = OrderedDict()          # leader tuple -> OrderedDict(follower tuple -> None), LRU first

    def insert(self, L, F):
        L, F = tuple(int(x) for x in L), tuple(int(x) for x in F)
        if L in self.t:
            self.t.move_to_end(L)
            fs = self.t[L]
            if F in fs:
                if self.refresh:
                    fs.move_to_end(F)
            else:
                if len(fs) == self.FC:
                    fs.popitem(last=False)
                fs[F] = None
        else:
            if len(self.t) == self.LC:
                self.t.popitem(last=False)
            self.t[L] = OrderedDict([(F, None)])

    def query(self, L):
        L = tuple(int(x) for x in L)
        if L not in self.t:
            return []
        self.t.move_to_end(L)
        return list(reversed(self.t[L].keys()))

    def peek(self, L):
        L = tuple(int(x) for x in L)
        return list(reversed(self.t[L].keys())) if L in self.t else []

    def update(self, s, n_old, n_new):
        w = self.LL + self.FL
        for i in range(max(0, n_old - w + 1), n_new - w + 1):
            self.insert(s[i:i + self.LL], s[i + self.LL:i + w])

    def dump(self):
        return [(L, list(fs.keys())) for L, fs in self.t.items()]
