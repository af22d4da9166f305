"""TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.

Plain restatement of the cost side of a transition, for the tests to hold the library against:
the transition estimate (Section 6: a function of bytes moved, link bandwidth and communicator set-up), the
profitability gate (Eq. 2, Section 4.3) and the horizon H_x (an exponential moving average of the intervals
between threshold crossings, one step before the first interval; Section 4.3).  The averaging weight is not
in the paper; it is a parameter here too."""
import math


def estimate_seconds(bytes_read: int, bytes_written: int, gbytes_per_s: float, setup_seconds: float) -> float:
    return setup_seconds + (bytes_read + bytes_written) / (gbytes_per_s * 1e9)


def payback_steps(l_tran: float, l_step_current: float, l_step_target: float) -> float:
    delta_l = l_step_current - l_step_target
    return l_tran / delta_l if delta_l > 0 else math.inf


def admit(l_tran, l_step_current, l_step_target, gamma, h_x, urgent=False) -> bool:
    """Eq. 2: delta_l > 0 and l_tran / delta_l <= gamma * h_x; the urgent path waives profitability; gamma = 0
    admits only urgent transitions."""
    if urgent:
        return True
    if gamma == 0:
        return False
    delta_l = l_step_current - l_step_target
    return delta_l > 0 and l_tran / delta_l <= gamma * h_x


class Horizon:
    def __init__(self, weight=0.5):
        self.h, self.weight, self.n = 1.0, weight, 0

    def crossing(self, interval_steps):
        self.h = interval_steps if self.n == 0 else (1 - self.weight) * self.h + self.weight * interval_steps
        self.n += 1
        return self.h
