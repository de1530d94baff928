"""The paper's analytical per-window timing model (Sec. 4, Eq. 3 and Eq. 4), as a small calculator.

Steady state: diffusion (d, with its launch overhead w_d) is on the critical path; VAE decode plus anchor
encode (v + a) and the next window's conditioning encode (w_e + e) overlap on separate streams, so a window
costs the diffusion path plus the LONGER of the two VAE branches.  Real time requires that to stay within the
budget of one window of new frames, T_rt = stride / fps (Sec. 3.3: 24 new frames at 24 fps = 1000 ms).
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class WindowTerms:
    """Per-window terms in milliseconds (names as in the paper's Sec. 4)."""
    w_d: float  # Python + kernel-launch overhead around diffusion
    d: float    # the four transformer forwards
    v: float    # split-VAE decode
    a: float    # anchor encode (serial after v on the decode stream)
    e: float    # next window's conditioning encode
    w_e: float  # extra wait on the encode stream beyond e

    def diffusion_path(self) -> float:
        return self.w_d + self.d

    def vae_path(self) -> float:
        return max(self.v + self.a, self.w_e + self.e)

    def window_ms(self) -> float:
        """Eq. 3: T_win ~ (w_d + d) + max(v + a, w_e + e)."""
        return self.diffusion_path() + self.vae_path()

    def serial_ms(self) -> float:
        """What the same terms would cost without the stream overlap."""
        return self.w_d + self.d + self.v + self.a + self.w_e + self.e


def realtime_budget_ms(stride_frames: int = 24, fps: float = 24.0) -> float:
    """Budget of one window: the time its new frames last when played (Sec. 3.3)."""
    return 1000.0 * stride_frames / fps


def feasible(terms: WindowTerms, budget_ms: float = 1000.0) -> bool:
    """Eq. 4: (w_d + d) + max(v + a, w_e + e) <= T_rt."""
    return terms.window_ms() <= budget_ms


def with_attention_ms(terms: WindowTerms, attention_ms_old: float, attention_ms_new: float) -> WindowTerms:
    """Replaces the attention share of d (e.g. by the attention milliseconds per window this library measures)."""
    return WindowTerms(terms.w_d, terms.d - attention_ms_old + attention_ms_new, terms.v, terms.a, terms.e, terms.w_e)


PAPER_TABLE_4 = WindowTerms(w_d=78.0, d=435.0, v=399.0, a=60.0, e=301.0, w_e=157.0)
