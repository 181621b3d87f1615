"""Seeded synthetic inputs for the LSAM workloads (numpy only; no optimiser arithmetic lives here).

The paper trains image classifiers on SVHN / CIFAR-10 / CIFAR-100; those datasets are not used.
These generators produce inputs with the same shapes (flattened 3x32x32 or 28x28 images, 10 / 100 /
1000 classes, tens of thousands of samples) whose values are Gaussian mixtures, plus the
least-squares problem and the flat gradient buffers of the optimiser-only sweep.
The same arrays are handed to the CUDA library and to the CPU oracle.
"""
import numpy as np


def least_squares_data(n_samples=4096, n_features=256, noise=0.01, seed=0):
    """X ~ N(0,1), w* ~ N(0,1), y = X w* + noise * N(0,1).  Returns (X fp32, y fp32, w_star fp32)."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n_samples, n_features), dtype=np.float32)
    w_star = rng.standard_normal(n_features, dtype=np.float32)
    y = (X.astype(np.float64) @ w_star.astype(np.float64) + noise * rng.standard_normal(n_samples)).astype(np.float32)
    return X, y, w_star


def gaussian_mixture(n_samples, n_features, n_classes, seed=0, chunk=8192):
    """Class means ~ N(0, I); sample i has label i mod n_classes and value mean[label] + N(0, I)."""
    rng = np.random.default_rng(seed)
    means = rng.standard_normal((n_classes, n_features), dtype=np.float32)
    labels = (np.arange(n_samples, dtype=np.int64) % n_classes).astype(np.int32)
    X = np.empty((n_samples, n_features), dtype=np.float32)
    for s in range(0, n_samples, chunk):
        e = min(s + chunk, n_samples)
        X[s:e] = rng.standard_normal((e - s, n_features), dtype=np.float32)
        X[s:e] += means[labels[s:e]]
    return X, labels


def mlp_param_count(widths):
    return int(sum(widths[l] * widths[l + 1] + widths[l + 1] for l in range(len(widths) - 1)))


def mlp_init(widths, seed=0):
    """One replica's flat vector: per layer W [out, in] ~ N(0, 2/in) row-major, then b = 0."""
    rng = np.random.default_rng(seed + 7919)
    parts = []
    for l in range(len(widths) - 1):
        fan_in, fan_out = widths[l], widths[l + 1]
        W = rng.standard_normal((fan_out, fan_in), dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
        parts.append(W.reshape(-1))
        parts.append(np.zeros(fan_out, dtype=np.float32))
    return np.concatenate(parts)


def cnn_dense_in(channels, img_h, img_w):
    """Features entering the first dense layer: the last channel count times the image size after one 2x2 pooling per convolution."""
    n_conv = len(channels) - 1
    return channels[-1] * (img_h >> n_conv) * (img_w >> n_conv)


def cnn_param_count(channels, dense, img_h, img_w):
    n = sum(channels[l + 1] * channels[l] * 9 + channels[l + 1] for l in range(len(channels) - 1))
    return int(n + mlp_param_count([cnn_dense_in(channels, img_h, img_w)] + list(dense)))


def cnn_init(channels, dense, img_h, img_w, seed=0):
    """Flat vector of the convolutional model: per convolution W [Cout, Cin * 9] ~ N(0, 2 / (9 Cin)) then b = 0, then the dense layers as in mlp_init."""
    rng = np.random.default_rng(seed + 15485863)
    parts = []
    for l in range(len(channels) - 1):
        fan_in = channels[l] * 9
        parts.append((rng.standard_normal((channels[l + 1], fan_in), dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))).reshape(-1))
        parts.append(np.zeros(channels[l + 1], dtype=np.float32))
    parts.append(mlp_init([cnn_dense_in(channels, img_h, img_w)] + list(dense), seed=seed))
    return np.concatenate(parts)


def replicate(x, K, jitter=0.0, seed=0):
    """Stack one vector K times ([K, d]); jitter > 0 adds N(0, jitter^2) so that replicas start apart."""
    out = np.repeat(np.asarray(x, dtype=np.float32)[None, :], K, axis=0).copy()
    if jitter > 0.0:
        rng = np.random.default_rng(seed + 104729)
        out += np.float32(jitter) * rng.standard_normal(out.shape, dtype=np.float32)
    return out


def flat_problem(K, d, seed=0, grad_std=0.1):
    """Optimiser-only sweep: x0 ~ N(0,1) [K, d]; g1, g2 ~ N(0, grad_std^2) [K, d]; centre = mean of x0."""
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal((K, d), dtype=np.float32)
    g1 = rng.standard_normal((K, d), dtype=np.float32) * np.float32(grad_std)
    g2 = rng.standard_normal((K, d), dtype=np.float32) * np.float32(grad_std)
    y0 = x0.astype(np.float64).mean(axis=0).astype(np.float32)
    return x0, y0, g1, g2
