"""I/O-aware verification-width controller, as plain Python (Section 4.2).

TEST INFRASTRUCTURE ONLY (see the package docstring).

q* = argmin_q T_round(q) / U(q) over the candidate widths.  Where the paper gives no formula
the same readings as the library are used and listed here so they can be checked by eye:
running means are exponential moving averages (first observation taken as is); the
verification cost is max(t_transfer, t_compute) (overlapped time counted once); every width is
tried `sample_rounds` times, in list order, before estimates are trusted; afterwards the width
changes only if best_cost < current_cost * (1 - switch_threshold); ties keep the smaller width.
"""


class WidthController:
    def __init__(self, widths, sample_rounds, switch_threshold, ema):
        self.widths = list(widths)
        self.sample_rounds = sample_rounds
        self.thr = switch_threshold
        self.ema = ema
        self.stats = {q: dict(n=0, draft=0.0, verify=0.0, other=0.0, u=0.0) for q in self.widths}
        self.current = self.widths[0]

    def observe(self, q, t_draft, t_transfer, t_compute, t_other, committed):
        s = self.stats[q]
        a = 1.0 if s["n"] == 0 else self.ema
        s["draft"] += a * (t_draft - s["draft"])
        s["verify"] += a * (max(t_transfer, t_compute) - s["verify"])
        s["other"] += a * (t_other - s["other"])
        s["u"] += a * (committed - s["u"])
        s["n"] += 1

    def cost(self, q):
        s = self.stats[q]
        return (s["draft"] + s["verify"] + s["other"]) / s["u"] if s["u"] > 0 else 1e300

    def next(self):
        for q in self.widths:
            if self.stats[q]["n"] < self.sample_rounds:
                self.current = q
                return q
        best = self.widths[0]
        for q in self.widths[1:]:
            if self.cost(q) < self.cost(best) or (self.cost(q) == self.cost(best) and q < best):
                best = q
        if best != self.current and self.cost(best) < self.cost(self.current) * (1.0 - self.thr):
            self.current = best
        return self.current
