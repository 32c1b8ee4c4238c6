"""Closed-form memory and cost models of the paper, restated for the unit tests.

TEST INFRASTRUCTURE ONLY.  Sec. 3.3 (memory analysis) counts stored scalars per
layer with the batch dimension left out; App. B (decoding-time complexity)
counts multiply-adds per cached token after removing the common factor L_t.
"""
import math


def memory_full(s, L, Dp):
    """Sec. 3.3, first equation: keys and values of s sinks and L non-sink tokens."""
    return 2 * (s + L) * Dp


def memory_s4r(s, L, Dp, r, G, W):
    """Sec. 3.3, second equation: sinks + both coefficient caches + query-coefficient window + both bases."""
    return 2 * s * Dp + 2 * L * r + G * W * r + 2 * Dp * r


def memory_ratio(s, L, Dp, r, G, W):
    """Sec. 3.3, third equation (persistent memory ratio)."""
    return (s * Dp + L * r + 0.5 * G * W * r + Dp * r) / ((s + L) * Dp)


def reconstructed_tokens(W, rho, L):
    """Sec. 3.3 / App. B: m_t = W + max(floor(rho L) - W, 0) = max(W, floor(rho L))."""
    return W + max(math.floor(rho * L) - W, 0)


def top_k_from_ratio(rho, L, W):
    """Eq. 14's budget: k = max(floor(rho L) - W, 0)."""
    return max(math.floor(rho * L) - W, 0)


def cost_full_reconstruction(r, Dp, G):
    """App. B: per-token coefficient of full reconstruction, r D' + G D'."""
    return r * Dp + G * Dp


def cost_s4r(r, Dp, G, W, rho):
    """App. B: per-token coefficients of S4R: (latent scoring, sparse reconstruction, sparse attention)."""
    return G * W * r, rho * r * Dp, rho * G * Dp
