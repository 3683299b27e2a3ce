"""UniGist gist-masked attention for B200 (sm_100a): Python binding of the C-ABI library."""
